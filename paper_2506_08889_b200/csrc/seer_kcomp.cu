// K compression cache update (Eq. 1b; Sec. 3.2): per block, max/min/mean pooling of the
// pre-RoPE keys over the block's rows, projection by W_k, RoPE at the block's first token,
// bf16 store.  Two kernels: the per-step append of the one block that has just filled, and the
// bulk build over many blocks after prefill.
#include "seer_device.cuh"
#include "seer_internal.h"

namespace seer {

namespace {

constexpr int kKcThreads = 256;
constexpr int kKcWarps = kKcThreads / 32;
constexpr int kInChunks = 3 * kHeadDim / 8;          // 48 pieces of 16 B per W_k row

// Append: grid (1, B*Hkv, row splits).  One block per (sequence, KV head); the output rows are
// split over gridDim.z CTAs so that the one block's latency chain is short.  Every warp owns
// rotary pairs (c, c + d_gate/2), two at a time: their four W_k rows are requested before the
// pooling starts.  (NB is the number of blocks per CTA; only NB = 1 is instantiated.)
template <int NB>
__device__ __forceinline__ void kcomp_body(const KcompParams& p) {
    __shared__ float red[kKcWarps][3][kHeadDim];                   // per-warp pooled partials
    __shared__ __align__(16) float feat[NB][3 * kHeadDim];         // [max | min | avg]

    const int u = blockIdx.y, i = u / p.num_kv_heads, h = u % p.num_kv_heads;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = p.block_size;
    const int half = p.d_gate / 2;
    const int pps = half / gridDim.z;                 // rotary pairs per row split
    const int pair_base = blockIdx.z * pps;

    // first batch of W_k rows, requested before the pooling starts
    uint4 wv[4][2];
    auto load_rows = [&](int pb) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int c = min(pair_base + pb + (k & 1), half - 1);
            const int r = c + (k >> 1) * half;
            const uint4* wrow = reinterpret_cast<const uint4*>(p.w_k + ((size_t)h * p.d_gate + r) * 3 * kHeadDim);
            wv[k][0] = __ldg(wrow + lane);
            wv[k][1] = lane < 16 ? __ldg(wrow + 32 + lane) : make_uint4(0u, 0u, 0u, 0u);
        }
    };
    load_rows(warp * 2);

    const int L = p.seq_lens[i];
    const int complete = L > 0 ? L / b : 0;           // blocks with all b rows present
    int nb = 0;                                       // blocks this CTA really handles
    int j_first;
    if (p.first_block < 0) {
        // the sequence has just grown by -first_block tokens: the block whose last row is among them
        j_first = complete - 1;
        nb = (blockIdx.x == 0 && complete > 0 && L % b < -p.first_block && j_first < p.max_blocks) ? 1 : 0;
    } else {
        j_first = p.first_block + blockIdx.x * NB;
        const int j_end = min(min(p.first_block + p.num_blocks, complete), p.max_blocks);
        nb = max(0, min(NB, j_end - j_first));
    }
    if (nb == 0) return;

    const size_t base = (size_t)i * p.stride_batch + (size_t)h * p.stride_head;
    const int cchunk = tid & 15;                      // 8 channels per thread
    const int rgrp = tid >> 4;                        // 16 row groups

    for (int q = 0; q < nb; ++q) {
        const int j = j_first + q;
        const size_t row0 = p.rows_block_local ? 0 : (size_t)j * b;
        float mx[8], mn[8], sm[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) { mx[c] = -INFINITY; mn[c] = INFINITY; sm[c] = 0.f; }
#pragma unroll 4
        for (int r = rgrp; r < b; r += 16) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(
                p.k_nope + base + (row0 + r) * p.stride_token + 8 * cchunk));
            const __nv_bfloat162* hh = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float2 f = bf16x2_to_float2(hh[c]);
                mx[2 * c] = fmaxf(mx[2 * c], f.x); mx[2 * c + 1] = fmaxf(mx[2 * c + 1], f.y);
                mn[2 * c] = fminf(mn[2 * c], f.x); mn[2 * c + 1] = fminf(mn[2 * c + 1], f.y);
                sm[2 * c] += f.x; sm[2 * c + 1] += f.y;
            }
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) {                 // the two row groups of a warp
            mx[c] = fmaxf(mx[c], __shfl_xor_sync(0xffffffffu, mx[c], 16));
            mn[c] = fminf(mn[c], __shfl_xor_sync(0xffffffffu, mn[c], 16));
            sm[c] += __shfl_xor_sync(0xffffffffu, sm[c], 16);
        }
        if (lane < 16) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                red[warp][0][8 * cchunk + c] = mx[c];
                red[warp][1][8 * cchunk + c] = mn[c];
                red[warp][2][8 * cchunk + c] = sm[c];
            }
        }
        __syncthreads();
        if (tid < kHeadDim) {
            float a = -INFINITY, m2 = INFINITY, s = 0.f;
#pragma unroll
            for (int w2 = 0; w2 < kKcWarps; ++w2) {
                a = fmaxf(a, red[w2][0][tid]);
                m2 = fminf(m2, red[w2][1][tid]);
                s += red[w2][2][tid];
            }
            feat[q][tid] = a;
            feat[q][kHeadDim + tid] = m2;
            feat[q][2 * kHeadDim + tid] = s / (float)b;
        }
        __syncthreads();
    }
    for (int q = nb; q < NB; ++q)
        for (int c = tid; c < 3 * kHeadDim; c += kKcThreads) feat[q][c] = 0.f;
    __syncthreads();

    // this lane's pieces of the features, all blocks (reused by every row)
    float fr[2][NB][8];
#pragma unroll
    for (int part = 0; part < 2; ++part) {
        const int ch = lane + 32 * part;
#pragma unroll
        for (int q = 0; q < NB; ++q)
#pragma unroll
            for (int c = 0; c < 8; ++c) fr[part][q][c] = ch < kInChunks ? feat[q][8 * ch + c] : 0.f;
    }

    for (int pb = warp * 2; pb < pps; pb += kKcWarps * 2) {
        float acc[4][NB];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
#pragma unroll
            for (int q = 0; q < NB; ++q) acc[k][q] = 0.f;
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                const __nv_bfloat162* hh = reinterpret_cast<const __nv_bfloat162*>(&wv[k][part]);
                float wf[8];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float2 f = bf16x2_to_float2(hh[c]);
                    wf[2 * c] = f.x; wf[2 * c + 1] = f.y;
                }
#pragma unroll
                for (int q = 0; q < NB; ++q) {
                    float a = acc[k][q];
#pragma unroll
                    for (int c = 0; c < 8; ++c) a = fmaf(wf[c], fr[part][q][c], a);
                    acc[k][q] = a;
                }
            }
        }
        if (pb + kKcWarps * 2 < pps) load_rows(pb + kKcWarps * 2);     // next batch on its way
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
            for (int q = 0; q < NB; ++q)
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) acc[k][q] += __shfl_xor_sync(0xffffffffu, acc[k][q], off);
        // RoPE at the position of the block's first token, then the bf16 store:
        // lane (2q + e) finishes pair e of block q
        if (lane < 2 * NB) {
            const int q = lane >> 1, e = lane & 1;
            const int c = pair_base + pb + e;
            if (q < nb && pb + e < pps) {
                float a = 0.f, bb = 0.f;
#pragma unroll
                for (int qq = 0; qq < NB; ++qq) {
                    if (qq == q) {
                        a = e ? acc[1][qq] : acc[0][qq];
                        bb = e ? acc[3][qq] : acc[2][qq];
                    }
                }
                const int j = j_first + q;
                float sn, cs;
                rope_sincos((double)j * (double)b, p.inv_freq[c], &sn, &cs);
                __nv_bfloat16* dst = p.kcomp + ((size_t)u * p.max_blocks + j) * p.d_gate;
                dst[c] = __float2bfloat16(a * cs - bb * sn);
                dst[c + half] = __float2bfloat16(bb * cs + a * sn);
            }
        }
    }
}

// The kernel normally waits for its predecessor in the stream before it touches memory.  As the last
// kernel of a decode step (p.wait_at_end) its inputs -- the keys the caller wrote before the step --
// are final from the start and nothing in the step reads the entry it writes, so it works at once, under
// the tail of the attention kernel before it, and waits for that kernel only before it ends: its own
// completion then still implies that of everything before it in the stream.
template <int NB>
__global__ void __launch_bounds__(kKcThreads) kcomp_kernel(const KcompParams p) {
    if (!p.wait_at_end) pdl_wait();
    pdl_launch_dependents();
    kcomp_body<NB>(p);
    if (p.wait_at_end) pdl_wait();
}

// ---- bulk build (after prefill): 16 consecutive blocks of one (sequence, KV head) per CTA --------
// Phase 1 streams the blocks' rows with many loads in flight (each warp pools two blocks) and
// leaves the 3*128 pooled features of every block in shared memory as bf16 (max and min are bf16
// values already; the mean is kept as a bf16 high part plus a bf16 correction, so nothing is
// lost).  Phase 2 is the contraction Y[row][block] = W_k[row][:] . feat[block][:] on the tensor
// cores (mma.sync m16n8k16: W_k rows on M straight from global memory, the 16 blocks on N);
// phase 3 rotates and stores.  Several CTAs share an SM, so one CTA's projection overlaps the
// others' streaming.
constexpr int kBulkBlocks = 16;
constexpr int kFeatStride = 3 * kHeadDim + 8;         // bf16 per block row (+8: conflict-free fragment reads)
constexpr int kLoStride = kHeadDim + 8;

__global__ void __launch_bounds__(kKcThreads, 4) kcomp_bulk_kernel(const KcompParams p) {
    __shared__ __align__(16) __nv_bfloat16 feat_hi[kBulkBlocks][kFeatStride];   // [max | min | avg]
    __shared__ __align__(16) __nv_bfloat16 feat_lo[kBulkBlocks][kLoStride];     // avg - bf16(avg)
    __shared__ float ybuf[kBulkBlocks][kMaxDGate];
    pdl_wait();
    pdl_launch_dependents();
    const int u = blockIdx.y, i = u / p.num_kv_heads, h = u % p.num_kv_heads;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = p.block_size;
    const int L = p.seq_lens[i];
    const int complete = L > 0 ? L / b : 0;
    const int j_first = p.first_block + blockIdx.x * kBulkBlocks;
    const int j_end = min(min(p.first_block + p.num_blocks, complete), p.max_blocks);
    const int nb = max(0, min(kBulkBlocks, j_end - j_first));
    if (nb == 0) return;
    const size_t base = (size_t)i * p.stride_batch + (size_t)h * p.stride_head;
    const int cchunk = lane & 15, rsel = lane >> 4;

    for (int q = warp; q < kBulkBlocks; q += kKcWarps) {
        // max and min stay packed bf16 pairs (they are bf16 values anyway), the sum is fp32
        __nv_bfloat162 mx[4], mn[4];
        float sm[8];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            mx[c] = __float2bfloat162_rn(-INFINITY);
            mn[c] = __float2bfloat162_rn(INFINITY);
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) sm[c] = 0.f;
        if (q < nb) {
            const __nv_bfloat16* src = p.k_nope + base + (size_t)(j_first + q) * b * p.stride_token + 8 * cchunk;
            // 16 rows per lane (32 rows of the block, 8 KiB per warp) are requested before any is looked at: the
            // kernel lives on the bytes it has in flight
            constexpr int kInFlight = 8;
            for (int r0 = 0; r0 < b; r0 += 2 * kInFlight) {
                uint4 buf[kInFlight];
#pragma unroll
                for (int k = 0; k < kInFlight; ++k) {
                    const int r = r0 + 2 * k + rsel;
                    buf[k] = r < b ? __ldg(reinterpret_cast<const uint4*>(src + (size_t)r * p.stride_token))
                                   : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int k = 0; k < kInFlight; ++k) {
                    if (r0 + 2 * k + rsel < b) {
                        const __nv_bfloat162* hh = reinterpret_cast<const __nv_bfloat162*>(&buf[k]);
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            mx[c] = __hmax2(mx[c], hh[c]);
                            mn[c] = __hmin2(mn[c], hh[c]);
                            const float2 f = bf16x2_to_float2(hh[c]);
                            sm[2 * c] += f.x; sm[2 * c + 1] += f.y;
                        }
                    }
                }
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t xm = *reinterpret_cast<uint32_t*>(&mx[c]), xn = *reinterpret_cast<uint32_t*>(&mn[c]);
                uint32_t ym = __shfl_xor_sync(0xffffffffu, xm, 16), yn = __shfl_xor_sync(0xffffffffu, xn, 16);
                mx[c] = __hmax2(mx[c], *reinterpret_cast<__nv_bfloat162*>(&ym));
                mn[c] = __hmin2(mn[c], *reinterpret_cast<__nv_bfloat162*>(&yn));
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) sm[c] += __shfl_xor_sync(0xffffffffu, sm[c], 16);
        }
        if (lane < 16) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const __nv_bfloat162 zero = __float2bfloat162_rn(0.f);
                *reinterpret_cast<__nv_bfloat162*>(&feat_hi[q][8 * cchunk + 2 * c]) = q < nb ? mx[c] : zero;
                *reinterpret_cast<__nv_bfloat162*>(&feat_hi[q][kHeadDim + 8 * cchunk + 2 * c]) = q < nb ? mn[c] : zero;
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float av = q < nb ? sm[c] / (float)b : 0.f;
                const __nv_bfloat16 av_hi = __float2bfloat16(av);
                feat_hi[q][2 * kHeadDim + 8 * cchunk + c] = av_hi;
                feat_lo[q][8 * cchunk + c] = __float2bfloat16(av - __bfloat162float(av_hi));
            }
        }
    }
    __syncthreads();

    // Y[row][block]: warp w takes output rows 16*mt .. +15 for mt = w, w+8, ...
    const int g = lane >> 2, t4 = lane & 3;
    for (int mt = warp; mt < p.d_gate / 16; mt += kKcWarps) {
        const uint32_t* w0 = reinterpret_cast<const uint32_t*>(p.w_k + ((size_t)h * p.d_gate + 16 * mt + g) * 3 * kHeadDim);
        const uint32_t* w1 = w0 + 8 * (3 * kHeadDim / 2);     // row + 8
        float acc[2][4];
#pragma unroll
        for (int n = 0; n < 2; ++n)
#pragma unroll
            for (int x = 0; x < 4; ++x) acc[n][x] = 0.f;
#pragma unroll 6
        for (int ks = 0; ks < 3 * kHeadDim / 16; ++ks) {
            uint32_t a[4];
            a[0] = __ldg(w0 + 8 * ks + t4);
            a[1] = __ldg(w1 + 8 * ks + t4);
            a[2] = __ldg(w0 + 8 * ks + 4 + t4);
            a[3] = __ldg(w1 + 8 * ks + 4 + t4);
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                const __nv_bfloat16* fr = &feat_hi[8 * n + g][16 * ks + 2 * t4];
                const uint32_t b0 = *reinterpret_cast<const uint32_t*>(fr);
                const uint32_t b1 = *reinterpret_cast<const uint32_t*>(fr + 8);
                mma_bf16_16816(acc[n], a, b0, b1);
                if (ks >= 2 * kHeadDim / 16) {        // the mean's correction term
                    const __nv_bfloat16* fl = &feat_lo[8 * n + g][16 * ks - 2 * kHeadDim + 2 * t4];
                    mma_bf16_16816(acc[n], a, *reinterpret_cast<const uint32_t*>(fl),
                                   *reinterpret_cast<const uint32_t*>(fl + 8));
                }
            }
        }
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            ybuf[8 * n + 2 * t4][16 * mt + g] = acc[n][0];
            ybuf[8 * n + 2 * t4 + 1][16 * mt + g] = acc[n][1];
            ybuf[8 * n + 2 * t4][16 * mt + g + 8] = acc[n][2];
            ybuf[8 * n + 2 * t4 + 1][16 * mt + g + 8] = acc[n][3];
        }
    }
    __syncthreads();

    const int half = p.d_gate / 2;
    for (int x = tid; x < nb * half; x += kKcThreads) {
        const int q = x / half, c = x % half;
        const int j = j_first + q;
        float sn, cs;
        rope_sincos((double)j * (double)b, p.inv_freq[c], &sn, &cs);
        const float a = ybuf[q][c], bb = ybuf[q][c + half];
        __nv_bfloat16* dst = p.kcomp + ((size_t)u * p.max_blocks + j) * p.d_gate;
        dst[c] = __float2bfloat16(a * cs - bb * sn);
        dst[c + half] = __float2bfloat16(bb * cs + a * sn);
    }
}


// ---- bulk build, streaming variant (b = 64, d_gate <= 128) ----------------------------------------
// One persistent CTA per SM, four kinds of warps that meet only through mbarriers:
//   producer (1 warp)    keeps a ring of 64-row stages (one block, 16 KiB) full with tiled copies, so
//                        the bytes in flight do not depend on what the other warps are doing;
//   pooling (10 warps)   each takes one block at a time out of shared memory and leaves the block's
//                        3*128 features (bf16; the mean as high part + correction: 512 numbers) in one of
//                        two feature buffers, laid out as the tensor cores read a K-major operand;
//   MMA (1 warp)         once 16 blocks are pooled, one thread multiplies them in: Y (128 rows of W_k x 16
//                        blocks, fp32 in tensor memory) = W_k[h] (from tensor memory, where it stays while
//                        the CTA's items have the same head) . features^T, 32 tcgen05.mma of K = 16;
//   epilogue (4 warps)   thread r has row r of W_k and of Y: it puts its row of W_k[h] into tensor memory when
//                        the head changes, reads its 16 products, and the four warps rotate and store -
//                        while the pooling warps are already on the next item.
// An item is 16 consecutive blocks of one (sequence, KV head); items are numbered head-major and dealt
// round-robin, so a CTA changes head a handful of times per launch.
//
// A block comes in kStagesPerBlock stages (a stage is freed as soon as it has been read, and what is free
// is in flight again).  Block number n of a CTA (counted over all its items) is pooled by warp
// n % kPoolWarps and its stages live in ring slots (n * kStagesPerBlock + part) % kStreamStages;
// kStreamStages is a multiple of kStagesPerBlock * kPoolWarps, so a slot is always read by the same
// warp, which goes through its stages in order: a wait on a slot's barrier is then never more than one
// phase away from the barrier's own, which is what a parity wait needs to be unambiguous.  (With a
// block-of-the-item -> warp rule a fast warp could ask for a slot's next use before the slot's current use
// had landed for another warp, and the parity test would pass on stale data.)
constexpr int kStreamStages = 10;                      // 160 KiB in flight per SM
constexpr int kStreamRows = 64;                        // the block size this kernel is written for
constexpr int kStageRows = kKcompStageRows;
constexpr int kStagesPerBlock = kStreamRows / kStageRows;
constexpr int kStageBytes = kStageRows * kHeadDim * 2;
constexpr int kStreamDGate = 128;
constexpr int kLensCache = 2048;                       // sequences whose length is kept in shared memory
constexpr int kPoolWarps = 10;                       // with 4 + 1 + 1 others: 16 warps
constexpr int kProjWarps = 5;                        // warps 0..3 epilogue, 4 MMA
constexpr int kEpiWarps = 4, kEpiThreads = 128;
constexpr int kFeatBytes = 8 * kBulkBlocks * 128;      // one feature buffer
constexpr int kKcTmemCols = 512;                       // W_k 256 columns (512 bf16 per row), Y twice 16
constexpr int kStreamThreads = 32 * (kProjWarps + kPoolWarps + 1);
static_assert(kStreamStages <= 32, "one producer lane per ring slot");
static_assert(kStreamStages % (kStagesPerBlock * kPoolWarps) == 0,
              "a ring slot must always be read by the same pooling warp");

struct __align__(1024) StreamSmem {
    // a stage: channels 0..63 of its 32 rows (128 B per row, 16-byte pieces swizzled by row as the copy engine
    // lays them out), then channels 64..127
    unsigned char ring[kStreamStages][kStageBytes];
    // features of 16 blocks, twice: [8 slabs of 64 features][16 blocks][128 B], 16-byte pieces swizzled by
    // block (what a K-major operand with the 128-byte swizzle looks like); slabs: max 0-1, min 2-3, the mean's
    // high part 4-5, its correction 6-7
    unsigned char feat[2][kFeatBytes];
    float ybuf[kBulkBlocks][kStreamDGate];
    uint64_t full[kStreamStages], empty[kStreamStages];
    uint64_t feat_full[2], feat_empty[2];
    uint64_t y_full[2], y_free[2];       // the products of an even / odd item are complete / have been read
    uint64_t w_ready;                    // a head's W_k is in tensor memory
    uint64_t tmem_done;                  // the epilogue warps have made their last tensor-memory access
    uint32_t tmem_base;
    int lens[kLensCache];                                             // seq_lens, read once
};
static_assert(sizeof(StreamSmem) + 1024 <= 227 * 1024, "one CTA's shared memory");
static_assert(kStageBytes % 2048 == 0, "both halves of a stage start on a swizzle-pattern boundary");

#ifdef SEER_DECODE_TRACE
#define KC_T(var) const long long var = clock64()
#define KC_ACC(slot, t0, t1) tr[slot] += (unsigned long long)((t1) - (t0))
#else
#define KC_T(var)
#define KC_ACC(slot, t0, t1)
#endif

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }

__global__ void __launch_bounds__(kStreamThreads, 1)
kcomp_stream_kernel(const __grid_constant__ CUtensorMap map_k, const KcompParams p) {
    extern __shared__ unsigned char smem_raw[];
    StreamSmem& sm = *reinterpret_cast<StreamSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        for (int s = 0; s < kStreamStages; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], 1);
        }
        for (int f = 0; f < 2; ++f) {
            mbar_init(&sm.feat_full[f], kPoolWarps);
            mbar_init(&sm.feat_empty[f], 1);
            mbar_init(&sm.y_full[f], 1);
            mbar_init(&sm.y_free[f], kEpiWarps);
        }
        mbar_init(&sm.w_ready, kEpiWarps);
        mbar_init(&sm.tmem_done, kEpiWarps);
        mbar_fence_init();
    }
    if (warp == kEpiWarps) tmem_alloc(&sm.tmem_base, kKcTmemCols);
    tc_fence_before_sync();
    pdl_wait();
    pdl_launch_dependents();
    // A small load issued while the copies flood the memory system waits microseconds behind them: the
    // lengths are fetched once, before any copy is in flight.
    for (int x = tid; x < min(p.batch, kLensCache); x += kStreamThreads) sm.lens[x] = p.seq_lens[x];
    __syncthreads();
    tc_fence_after_sync();

    const int b = p.block_size;                        // == kStreamRows
    const int groups = (p.num_blocks + kBulkBlocks - 1) / kBulkBlocks;
    const int per_head = groups * p.batch;
    const int n_items = per_head * p.num_kv_heads;
    bool dead = false;                                 // a wait ran out: stop waiting, finish the motions
#ifdef SEER_DECODE_TRACE
    unsigned long long tr[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const long long t_begin = clock64();
#endif

    // item -> (head, sequence, first block) and the number of complete blocks of it that exist
    auto item_blocks = [&](int item, int& h, int& i, int& j_first) {
        h = item / per_head;
        const int rem = item - h * per_head;
        const int g = rem / p.batch;
        i = rem - g * p.batch;
        const int L = i < kLensCache ? sm.lens[i] : p.seq_lens[i];
        const int complete = L > 0 ? L / b : 0;
        j_first = p.first_block + g * kBulkBlocks;
        const int j_end = min(min(p.first_block + p.num_blocks, complete), p.max_blocks);
        return max(0, min(kBulkBlocks, j_end - j_first));
    };

    if (warp == kProjWarps + kPoolWarps) {
        // ---- producer ----
        // Lane l owns ring slot l: it walks the CTA's items for the stages l, l + kStreamStages, ... and
        // re-arms its slot the moment the slot is free.  The lanes poll in lockstep (one look at the slot's
        // barrier per turn, no waiting inside), so slots that are freed together are refilled together
        // instead of one barrier round trip after the other.
        if (lane == 0) tma_prefetch_desc(&map_k);
        uint32_t cursor = lane;                        // the stage this lane arms next
        uint32_t item_first = 0;                       // stage number of the first stage of `item`
        int item = blockIdx.x, h = 0, i = 0, j_first = 0;
        int nb = item < n_items ? item_blocks(item, h, i, j_first) : 0;
        uint32_t idle = 0;
        while (true) {
            while (item < n_items && cursor >= item_first + (uint32_t)(nb * kStagesPerBlock)) {
                item_first += nb * kStagesPerBlock;
                item += gridDim.x;
                nb = item < n_items ? item_blocks(item, h, i, j_first) : 0;
            }
            const bool have = lane < kStreamStages && item < n_items;
            if (!__any_sync(0xffffffffu, have)) break;
            const bool go = have && mbar_test_wait(&sm.empty[lane], ((cursor / kStreamStages) & 1u) ^ 1u);
            if (go) {
                const uint32_t rel = cursor - item_first;
                const int q = rel / kStagesPerBlock, part = rel % kStagesPerBlock;
                const int row0 = (j_first + q) * b + part * kStageRows;
                mbar_arrive_expect_tx(&sm.full[lane], kStageBytes);
                tma_load_4d(sm.ring[lane], &map_k, &sm.full[lane], 0, row0, h, i);
                tma_load_4d(sm.ring[lane] + kStageBytes / 2, &map_k, &sm.full[lane], 64, row0, h, i);
                cursor += kStreamStages;
            }
            const uint32_t went = __ballot_sync(0xffffffffu, go);
#ifdef SEER_DECODE_TRACE
            tr[0] += 1; tr[1] += __popc(went);
#endif
            if (went) {
                idle = 0;
            } else if (++idle > 64) {
                if (idle > (1u << 22)) {               // seconds: nothing will free these slots any more
                    raise_status(p.status, DEV_TIMEOUT);
                    break;
                }
                __nanosleep(32);
            }
        }
    } else if (warp >= kProjWarps) {
        // ---- pooling ----
        const int pw = warp - kProjWarps;
        const int cchunk = lane & 15;
        // where this lane's piece sits in rows 2k + (lane >> 4) for k = 0..3 mod 4 (see the read below)
        const int lane_off = (cchunk >> 3) * (kStageBytes / 2) + (lane >> 4) * 128;
        int piece_off[4];
#pragma unroll
        for (int m = 0; m < 4; ++m) piece_off[m] = (((cchunk & 7) ^ (lane >> 4)) ^ (2 * m)) << 4;
        uint32_t block_no = 0, n_done = 0;                 // blocks and items this CTA has been through
        for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
            int h, i, j_first;
            const int nb = item_blocks(item, h, i, j_first);
            if (nb == 0) continue;
            const int fb = n_done & 1;
            KC_T(t_fe0);
            if (!dead && !mbar_wait(&sm.feat_empty[fb], ((n_done >> 1) & 1u) ^ 1u, p.status)) dead = true;
            KC_T(t_fe1);
            KC_ACC(0, t_fe0, t_fe1);
            for (int q = 0; q < kBulkBlocks; ++q) {
                if ((block_no + q) % kPoolWarps != (uint32_t)pw) continue;
                __nv_bfloat162 mx[4], mn[4];
                float sum[8];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    mx[c] = __float2bfloat162_rn(-INFINITY);
                    mn[c] = __float2bfloat162_rn(INFINITY);
                }
#pragma unroll
                for (int c = 0; c < 8; ++c) sum[c] = 0.f;
                if (q < nb) {
#pragma unroll 1
                    for (int part = 0; part < kStagesPerBlock; ++part) {
                        const uint32_t sn = (block_no + q) * kStagesPerBlock + part;
                        const int s = sn % kStreamStages;
                        KC_T(t_w0);
                        if (!dead && !mbar_wait(&sm.full[s], (sn / kStreamStages) & 1u, p.status)) dead = true;
                        KC_T(t_w1);
                        KC_ACC(1, t_w0, t_w1);
                        // lane: 16-byte column piece (lane & 15) of rows 2k + (lane >> 4); piece c of row r of a
                        // 64-channel half sits at position c ^ (r & 7) of the row's 128 bytes
                        const unsigned char* st = sm.ring[s] + lane_off;
#pragma unroll 8
                        for (int k = 0; k < kStageRows / 2; ++k) {
                            const uint4 v = *reinterpret_cast<const uint4*>(st + k * 256 + piece_off[k & 3]);
                            const __nv_bfloat162* hh = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                mx[c] = __hmax2(mx[c], hh[c]);
                                mn[c] = __hmin2(mn[c], hh[c]);
                                const float2 f = bf16x2_to_float2(hh[c]);
                                sum[2 * c] += f.x; sum[2 * c + 1] += f.y;
                            }
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&sm.empty[s]);
                        KC_T(t_w2);
                        KC_ACC(2, t_w1, t_w2);
#ifdef SEER_DECODE_TRACE
                        tr[3] += 1;
#endif
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t xm = *reinterpret_cast<uint32_t*>(&mx[c]), xn = *reinterpret_cast<uint32_t*>(&mn[c]);
                        uint32_t ym = __shfl_xor_sync(0xffffffffu, xm, 16), yn = __shfl_xor_sync(0xffffffffu, xn, 16);
                        mx[c] = __hmax2(mx[c], *reinterpret_cast<__nv_bfloat162*>(&ym));
                        mn[c] = __hmin2(mn[c], *reinterpret_cast<__nv_bfloat162*>(&yn));
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c) sum[c] += __shfl_xor_sync(0xffffffffu, sum[c], 16);
                }
                if (lane < 16) {
                    // 8 features per kind and lane: one 16-byte piece each, at its swizzled place in row q of its slab
                    uint4 pmax = make_uint4(0u, 0u, 0u, 0u), pmin = pmax, phi = pmax, plo = pmax;
                    if (q < nb) {
                        pmax = make_uint4(*reinterpret_cast<uint32_t*>(&mx[0]), *reinterpret_cast<uint32_t*>(&mx[1]),
                                          *reinterpret_cast<uint32_t*>(&mx[2]), *reinterpret_cast<uint32_t*>(&mx[3]));
                        pmin = make_uint4(*reinterpret_cast<uint32_t*>(&mn[0]), *reinterpret_cast<uint32_t*>(&mn[1]),
                                          *reinterpret_cast<uint32_t*>(&mn[2]), *reinterpret_cast<uint32_t*>(&mn[3]));
                        uint32_t hi[4], lo[4];
#pragma unroll
                        for (int c = 0; c < 8; c += 2) {
                            const float a0 = sum[c] * (1.f / kStreamRows), a1 = sum[c + 1] * (1.f / kStreamRows);
                            const __nv_bfloat162 h2 = __floats2bfloat162_rn(a0, a1);
                            hi[c >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
                            const float2 hf = bf16x2_to_float2(h2);
                            lo[c >> 1] = pack_bf16x2(a0 - hf.x, a1 - hf.y);
                        }
                        phi = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                        plo = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                    }
                    unsigned char* f0 = sm.feat[fb] + (cchunk >> 3) * (kBulkBlocks * 128) + q * 128 + (((cchunk & 7) ^ (q & 7)) << 4);
                    *reinterpret_cast<uint4*>(f0) = pmax;
                    *reinterpret_cast<uint4*>(f0 + 2 * kBulkBlocks * 128) = pmin;
                    *reinterpret_cast<uint4*>(f0 + 4 * kBulkBlocks * 128) = phi;
                    *reinterpret_cast<uint4*>(f0 + 6 * kBulkBlocks * 128) = plo;
                }
            }
            block_no += nb;
            ++n_done;
            fence_proxy_async_smem();              // the tensor cores read the features through the asynchronous proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.feat_full[fb]);
#ifdef SEER_DECODE_TRACE
            { const long long t_e = clock64(); tr[4] += (unsigned long long)(t_e - t_fe0); }
#endif
        }
    } else if (warp == kEpiWarps) {
        // ---- MMA warp: Y = W_k[h] . features^T per item, issued by lane 0 ----
        const uint32_t tbase = sm.tmem_base;
        constexpr uint32_t idesc = tc_idesc_bf16(128, kBulkBlocks, false);
        int h_held = -1;
        uint32_t n_done = 0, n_heads = 0;
        for (int item = blockIdx.x; item < n_items && !dead; item += gridDim.x) {
            int h, i, j_first;
            const int nb = item_blocks(item, h, i, j_first);
            if (nb == 0) continue;
            if (h != h_held) {
                // the epilogue warps put the new head's rows in place (after the last products of the old one)
                if (!mbar_wait(&sm.w_ready, n_heads & 1u, p.status)) { dead = true; break; }
                ++n_heads;
                h_held = h;
            }
            const int fb = n_done & 1;
            if (!mbar_wait(&sm.feat_full[fb], (n_done >> 1) & 1u, p.status)) { dead = true; break; }
            // the Y buffer of two items ago has been read
            if (n_done >= 2 && !mbar_wait(&sm.y_free[fb], ((n_done - 2) >> 1) & 1u, p.status)) { dead = true; break; }
            __syncwarp();
            if (lane == 0) {
                tc_fence_after_sync();
                const uint64_t fd = tc_smem_desc(smem_u32(sm.feat[fb]), 16, 1024);
#pragma unroll 4
                for (int ks = 0; ks < 32; ++ks)
                    tc_mma_ts(tbase + 256 + 16 * fb, tbase + 8 * ks, fd + (uint64_t)(((ks >> 2) * (kBulkBlocks * 128) + (ks & 3) * 32) >> 4),
                              idesc, ks > 0);
                tc_commit(&sm.y_full[fb]);
                tc_commit(&sm.feat_empty[fb]);         // the features have been read
            }
            __syncwarp();
            ++n_done;
        }
        // the tensor memory goes back once the epilogue warps are done with it (or a wait has run out)
        mbar_wait(&sm.tmem_done, 0, p.status);
        __syncwarp();
        tmem_dealloc(tbase, kKcTmemCols);
    } else if (warp < kEpiWarps) {
        // ---- epilogue: W_k into tensor memory, products out of it, rotation, store ----
        const int r = tid;                            // row of W_k[h] and of Y, lane of tensor memory
        const uint32_t tbase = sm.tmem_base + ((uint32_t)(32 * warp) << 16);
        int h_held = -1;
        uint32_t n_done = 0;
        for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
            int h, i, j_first;
            const int nb = item_blocks(item, h, i, j_first);
            if (nb == 0) continue;
            if (h != h_held) {
                // (every product that used the old rows is complete: this thread has read the last of them)
                const uint4* wrow = reinterpret_cast<const uint4*>(p.w_k + ((size_t)h * p.d_gate + min(r, p.d_gate - 1)) * 3 * kHeadDim);
#pragma unroll 1
                for (int c0 = 0; c0 < 8; ++c0) {          // 8 x 32 columns = 512 bf16: [max | min | avg | avg again]
                    uint32_t wr[32];
                    const int src = (c0 < 6 ? c0 : c0 - 2) * 8;   // (16-byte pieces of the row; the mean's weights serve its correction too)
#pragma unroll
                    for (int x = 0; x < 8; ++x) {
                        const uint4 v = r < p.d_gate ? __ldg(wrow + src + x) : make_uint4(0u, 0u, 0u, 0u);
                        wr[4 * x] = v.x; wr[4 * x + 1] = v.y; wr[4 * x + 2] = v.z; wr[4 * x + 3] = v.w;
                    }
                    tmem_st32(tbase + 32 * c0, wr);
                }
                tmem_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.w_ready);
                h_held = h;
            }
            const int fb = n_done & 1;
            KC_T(t_p0);
            if (!dead && !mbar_wait(&sm.y_full[fb], (n_done >> 1) & 1u, p.status)) dead = true;
            KC_T(t_p1);
            KC_ACC(0, t_p0, t_p1);
            ++n_done;
            __syncwarp();
            tc_fence_after_sync();
            uint32_t y[16];
            tmem_ld16(tbase + 256 + 16 * fb, y);
            tmem_wait_ld();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.y_free[fb]);
#pragma unroll
            for (int q = 0; q < kBulkBlocks; ++q) sm.ybuf[q][r] = __uint_as_float(y[q]);
            epi_sync();
            const int half = p.d_gate / 2;
            const int u = i * p.num_kv_heads + h;
            // eight rotary pairs per thread: two 16-byte stores instead of sixteen 2-byte ones (a store, too,
            // queues behind the copies)
            for (int x = tid; x < nb * (half / 8); x += kEpiThreads) {
                const int q = x / (half / 8), c0 = 8 * (x % (half / 8));
                const int j = j_first + q;
                uint32_t lo[4], hi[4];
#pragma unroll
                for (int e = 0; e < 8; e += 2) {
                    float r0[2], r1[2];
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        float sn, cs;
                        rope_sincos((double)j * (double)b, p.inv_freq[c0 + e + k], &sn, &cs);
                        const float a = sm.ybuf[q][c0 + e + k], bb = sm.ybuf[q][c0 + e + k + half];
                        r0[k] = a * cs - bb * sn;
                        r1[k] = bb * cs + a * sn;
                    }
                    lo[e / 2] = pack_bf16x2(r0[0], r0[1]);
                    hi[e / 2] = pack_bf16x2(r1[0], r1[1]);
                }
                __nv_bfloat16* dst = p.kcomp + ((size_t)u * p.max_blocks + j) * p.d_gate + c0;
                *reinterpret_cast<uint4*>(dst) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                *reinterpret_cast<uint4*>(dst + half) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            }
            epi_sync();                                    // (the products' buffer is written again for the next item)
            KC_T(t_p2);
            KC_ACC(1, t_p1, t_p2);
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.tmem_done);
    }
#ifdef SEER_DECODE_TRACE
    if (lane == 0) {
        tr[7] = (unsigned long long)(clock64() - t_begin);
        for (int k = 0; k < 8; ++k) p.trace[((size_t)blockIdx.x * (kStreamThreads / 32) + warp) * 8 + k] = tr[k];
    }
#endif
}

}  // namespace

bool kcomp_bulk_streams(const KcompParams& p) {
    const int U = p.batch * p.num_kv_heads;
    const int gx = (p.num_blocks + kBulkBlocks - 1) / kBulkBlocks;
    return p.first_block >= 0 && p.block_size == kStreamRows && p.d_gate <= kStreamDGate && !p.rows_block_local &&
           (long long)gx * U >= 2LL * p.sm_count;
}

cudaError_t launch_kcomp_append(const KcompParams& p, const CUtensorMap* map_k, cudaStream_t stream, int* launched) {
    const int U = p.batch * p.num_kv_heads;
    *launched = 0;
    if (U <= 0) return cudaSuccess;
    if (p.first_block < 0) {
        // one block per unit: split the d_gate/2 rotary pairs over 4 CTAs (16, 8 or 32 pairs each)
        cudaError_t e = launch_pdl(kcomp_kernel<1>, dim3(1, U, 4), dim3(kKcThreads), 0, stream, p);
        *launched = 1;
        return e;
    } else {
        const int gx = (p.num_blocks + kBulkBlocks - 1) / kBulkBlocks;
        if (gx <= 0) return cudaSuccess;
        if (map_k && kcomp_bulk_streams(p)) {
            static bool attr_set[64] = {};
            int dev = 0;
            cudaError_t e = cudaGetDevice(&dev);
            if (e != cudaSuccess) return e;
            if (dev < 0 || dev >= 64 || !attr_set[dev]) {
                e = cudaFuncSetAttribute(kcomp_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(StreamSmem) + 1024);
                if (e != cudaSuccess) return e;
                if (dev >= 0 && dev < 64) attr_set[dev] = true;
            }
            e = launch_pdl(kcomp_stream_kernel, dim3(min(p.sm_count, gx * U), 1, 1), dim3(kStreamThreads),
                           sizeof(StreamSmem) + 1024, stream, *map_k, p);
            *launched = 1;
            return e;
        }
        cudaError_t e = launch_pdl(kcomp_bulk_kernel, dim3(gx, U, 1), dim3(kKcThreads), 0, stream, p);
        *launched = 1;
        return e;
    }
    *launched = 1;
    return cudaGetLastError();
}

}  // namespace seer
