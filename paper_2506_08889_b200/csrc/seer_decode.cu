// Split-KV flash decoding for GQA on sm_100a: the block-sparse kernel of Sec. 3.3 and the
// dense kernel built from the same parts.
//
// Work decomposition.  A "unit" is one (sequence, KV head) pair; its work is the list of
// 64-token tiles of its selected blocks (sparse) or of its whole sequence (dense).  All
// units' tile lists are laid end to end and cut into `gridDim.x` equal contiguous ranges,
// one per CTA, so every CTA streams the same number of KV bytes whatever the per-unit
// selection counts are.  A CTA whose range covers a unit completely writes the final
// output; otherwise it writes an un-normalised partial (o, max, sum) and takes a ticket;
// the CTA that draws the last ticket of a unit merges the partials (log-sum-exp combine).
// There is no spin-wait anywhere: the merge is done by whoever finishes last.
//
// Inside a CTA: one producer warp walks the range, turns each tile into TMA box loads
// (K and V, 2 x 64x64 bf16 boxes each, 128-byte swizzle) into a ring of shared-memory
// stages, and passes per-tile metadata beside the data.  Four consumer warps each own 16
// of a tile's 64 tokens and keep private online-softmax state (running max, sum, and the
// 128 x 8 output accumulator), so they never synchronise with each other inside the loop:
//     S^T (16 tok x 8 heads) = K_slice (16 x 128) . Q^T (128 x 8)      mma.sync m16n8k16
//     P^T -> bf16, transposed in registers (movmatrix) into the B operand
//     O^T (128 x 8)        += V_slice^T (128 x 16) . P^T (16 x 8)       mma.sync m16n8k16
// The g <= 8 query heads of the group sit on the MMA's N = 8 side, tokens on M.
#include "seer_device.cuh"
#include "seer_internal.h"

namespace seer {

namespace {

constexpr int kStages = 3;
constexpr int kConsumerWarps = 4;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kHalfTileBytes = kTileTokens * 128;          // 64 rows x 128 B (64 bf16 channels)
constexpr int kTileBytes = 2 * kHalfTileBytes;             // one K or V tile: 16 KiB
constexpr int kStageBytes = 2 * kTileBytes;                // K + V
constexpr int kMergeStride = 132;                          // floats per head row (bank spread)

struct StageMeta {
    int nvalid;        // tokens of this tile that exist (0 = nothing was loaded)
    int unit;          // (sequence, KV head) index
    int last;          // last tile of this CTA's piece of the unit
    int unit_first;    // global index of the unit's first tile
    int unit_tiles;    // tiles of the unit
};

struct __align__(1024) Smem {
    unsigned char stage[kStages][kStageBytes];
    float merge_o[kConsumerWarps - 1][kMaxGroup][kMergeStride];
    float merge_ml[2][kConsumerWarps][2][kMaxGroup];   // double-buffered by piece parity
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t merge_bar[2];
    StageMeta meta[kStages];
    int scan_warp[kThreads / 32];
    int start_unit;
    int start_off;
};

// Programmatic dependent launch: the kernel may start while its predecessor in the stream is
// still running; nothing the predecessor writes is read before pdl_wait().
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

#ifdef SEER_DECODE_TRACE
__device__ __forceinline__ void trace_stamp(const DecodeParams& p, int slot) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    p.trace[(size_t)blockIdx.x * 8 + slot] = t;
}
#define SEER_STAMP(slot) trace_stamp(p, slot)
#else
#define SEER_STAMP(slot) ((void)0)
#endif

template <bool SPARSE>
__device__ __forceinline__ int tiles_of(const DecodeParams& p, int u) {
    int L = p.seq_lens[u / p.num_kv_heads];
    if (L <= 0) return 0;
    if (SPARSE) {
        int c = p.block_cnt ? p.block_cnt[u] : p.max_sel;
        c = max(0, min(c, p.max_sel));
        return c * p.tiles_per_block;
    } else {
        int t = (L + kTileTokens - 1) / kTileTokens;
        return min(t, p.max_blocks_cap);
    }
}

// CTA that owns global tile t when T tiles are cut into G equal contiguous ranges
// (range c = [floor(c*T/G), floor((c+1)*T/G)) ).
__device__ __forceinline__ int cta_of(long long t, long long T, long long G) {
    return (int)(((t + 1) * G - 1) / T);
}

__device__ __forceinline__ void write_zero_unit(const DecodeParams& p, int u) {
    int i = u / p.num_kv_heads, h = u % p.num_kv_heads;
    for (int hh = 0; hh < p.group; ++hh) {
        size_t row = (size_t)i * p.num_q_heads + (size_t)h * p.group + hh;
        for (int c = 0; c < kHeadDim; ++c) p.out[row * kHeadDim + c] = __float2bfloat16(0.f);
        if (p.lse) p.lse[row] = -INFINITY;
    }
}

template <bool SPARSE, bool PAGED>
__global__ void __launch_bounds__(kThreads, 2)
decode_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
              const DecodeParams p) {
    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int U = p.num_units;
    const int cta = blockIdx.x;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], kConsumerWarps);
        }
        mbar_init(&sm.merge_bar[0], kConsumerWarps);
        mbar_init(&sm.merge_bar[1], kConsumerWarps);
        mbar_fence_init();
        sm.start_unit = U;
        sm.start_off = 0;
    }
    if (warp == kConsumerWarps && lane == 0) {
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
    }

    if (tid == 0) SEER_STAMP(0);
    pdl_wait();
    if (tid == 0) SEER_STAMP(1);

    // ---- every CTA sums the units' tile counts and finds where its own range starts ----
    const int per = (U + kThreads - 1) / kThreads;
    const int u_lo = min(U, tid * per), u_hi = min(U, u_lo + per);
    int mine = 0;
    for (int u = u_lo; u < u_hi; ++u) {
        int t = tiles_of<SPARSE>(p, u);
        if (t == 0 && cta == 0) write_zero_unit(p, u);   // units without work: zeros, -inf
        mine += t;
    }
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) sm.scan_warp[warp] = incl;
    __syncthreads();
    int warp_base = 0, T_i = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
        int v = sm.scan_warp[w];
        if (w < warp) warp_base += v;
        T_i += v;
    }
    const long long T = T_i;
    if (T == 0) return;
    // never more ranges than tiles: every range in use is non-empty, so a unit's pieces are
    // exactly the CTAs between the owners of its first and last tile
    const long long G = min((long long)gridDim.x, T);
    if (cta >= G) return;
    const int excl = warp_base + incl - mine;
    const int t_begin = (int)((cta * T) / G), t_end = (int)(((cta + 1) * T) / G);
    if (t_begin >= t_end) return;
    if (mine > 0 && excl <= t_begin && t_begin < excl + mine) {
        int acc = excl;
        for (int u = u_lo; u < u_hi; ++u) {
            int t = tiles_of<SPARSE>(p, u);
            if (t_begin < acc + t) {
                sm.start_unit = u;
                sm.start_off = t_begin - acc;
                break;
            }
            acc += t;
        }
    }
    __syncthreads();
    const int n_tiles = t_end - t_begin;
    if (tid == 0) SEER_STAMP(2);

    if (warp == kConsumerWarps) {
        // =========================== producer warp ====================================
        int cu = sm.start_unit, ce = sm.start_off;
        if (cu >= U) return;
        int cut = tiles_of<SPARSE>(p, cu);
        int cpu = t_begin - ce;
        int it = 0;
        for (int t = 0; t < n_tiles; t += 32) {
            const int n_chunk = min(32, n_tiles - t);
            // deal the next n_chunk tiles to lanes, walking over unit boundaries
            int my_u = -1, my_e = 0, my_ut = 0, my_pu = 0;
            int base = 0;
            while (base < n_chunk) {
                int avail = cut - ce;
                if (avail <= 0) {
                    cpu += cut;
                    ++cu;
                    ce = 0;
                    if (cu >= U) { cut = 0; break; }
                    cut = tiles_of<SPARSE>(p, cu);
                    continue;
                }
                int take = min(avail, n_chunk - base);
                if (lane >= base && lane < base + take) {
                    my_u = cu; my_e = ce + lane - base; my_ut = cut; my_pu = cpu;
                }
                base += take;
                ce += take;
            }
            // per-lane tile descriptor
            int nvalid = 0, row = 0, outer = 0, head = 0, last = 0;
            if (my_u >= 0) {
                const int i = my_u / p.num_kv_heads;
                head = my_u % p.num_kv_heads;
                const int L = p.seq_lens[i];
                int tok0 = 0;
                if (SPARSE) {
                    const int blk = p.block_idx[(size_t)my_u * p.max_sel + my_e / p.tiles_per_block];
                    const int n_i = (L + p.block_size - 1) / p.block_size;
                    if (blk >= n_i) raise_status(p.status, DEV_BAD_INDEX);
                    if (blk >= 0 && blk < n_i) {
                        tok0 = blk * p.block_size + (my_e % p.tiles_per_block) * kTileTokens;
                        nvalid = max(0, min(kTileTokens, L - tok0));
                    }
                } else {
                    tok0 = my_e * kTileTokens;
                    nvalid = max(0, min(kTileTokens, L - tok0));
                }
                if (PAGED) {
                    if (nvalid > 0) {
                        const int pg = p.page_table[(size_t)i * p.page_table_stride + tok0 / p.page_size];
                        if (pg < 0 || pg >= p.num_pages) {
                            raise_status(p.status, DEV_BAD_INDEX);
                            nvalid = 0;
                        }
                        outer = pg;
                        row = tok0 % p.page_size;
                    }
                } else {
                    outer = i;
                    row = tok0;
                }
                last = (my_e == my_ut - 1) || (t + lane == n_tiles - 1);
            } else if (lane < n_chunk) {
                // the counts changed under us: keep the pipeline protocol, load nothing
                my_u = 0; my_ut = 1; last = (t + lane == n_tiles - 1);
                raise_status(p.status, DEV_BAD_INDEX);
            }
            for (int s = 0; s < n_chunk; ++s, ++it) {
                const int s_nvalid = __shfl_sync(0xffffffffu, nvalid, s);
                const int s_row = __shfl_sync(0xffffffffu, row, s);
                const int s_outer = __shfl_sync(0xffffffffu, outer, s);
                const int s_head = __shfl_sync(0xffffffffu, head, s);
                const int s_last = __shfl_sync(0xffffffffu, last, s);
                const int s_u = __shfl_sync(0xffffffffu, my_u, s);
                const int s_pu = __shfl_sync(0xffffffffu, my_pu, s);
                const int s_ut = __shfl_sync(0xffffffffu, my_ut, s);
                if (lane == 0) {
                    const int st = it % kStages;
                    if (!mbar_wait(&sm.empty[st], ((it / kStages) & 1) ^ 1, p.status)) return;
                    sm.meta[st] = StageMeta{s_nvalid, s_u, s_last, s_pu, s_ut};
                    if (s_nvalid > 0) {
                        unsigned char* dst = sm.stage[st];
                        mbar_arrive_expect_tx(&sm.full[st], kStageBytes);
                        tma_load_4d(dst, &map_k, &sm.full[st], 0, s_row, s_head, s_outer);
                        tma_load_4d(dst + kHalfTileBytes, &map_k, &sm.full[st], 64, s_row, s_head, s_outer);
                        tma_load_4d(dst + kTileBytes, &map_v, &sm.full[st], 0, s_row, s_head, s_outer);
                        tma_load_4d(dst + kTileBytes + kHalfTileBytes, &map_v, &sm.full[st], 64, s_row,
                                    s_head, s_outer);
                    } else {
                        mbar_arrive(&sm.full[st]);
                    }
                    if (it == 0) SEER_STAMP(3);
                    if (it == n_tiles - 1) SEER_STAMP(4);
                }
            }
        }
        return;
    }

    // =============================== consumer warps =====================================
    const int w = warp;
    const int qd = lane & 3;            // column pair: heads 2*qd, 2*qd+1
    const int rw = lane >> 2;           // row within an 8-row slab
    uint32_t bq[8][2];                  // Q^T B-fragments for the 8 k-steps over d
    uint32_t bq_pre[8][2];              // the same for the unit expected next (prefetched)
    float o[8][4];                      // O^T accumulators: 8 m-tiles over d
    float m_run[2], l_run[2];
    int cur_unit = -1;
    int seg = 0;
    auto load_q = [&](uint32_t (&dst)[8][2], int unit) {
        const int i = unit / p.num_kv_heads, h = unit % p.num_kv_heads;
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
            p.q + ((size_t)i * p.num_q_heads + (size_t)h * p.group + rw) * kHeadDim);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            dst[ks][0] = (rw < p.group) ? __ldg(qrow + (16 * ks + 2 * qd) / 2) : 0u;
            dst[ks][1] = (rw < p.group) ? __ldg(qrow + (16 * ks + 8 + 2 * qd) / 2) : 0u;
        }
    };
    int pre_unit = sm.start_unit;       // requested now, long before the first tile lands
    if (pre_unit < U) load_q(bq_pre, pre_unit);

    // lane-constant parts of the ldmatrix addresses (swizzle: 16-B chunk ^= row & 7)
    const int k_row = 16 * w + ((lane >> 3) & 1) * 8 + (lane & 7);
    const int k_csel = lane >> 4;                    // which of the two 16-B chunks of a k-step
    const int v_row = 16 * w + ((lane >> 4) & 1) * 8 + (lane & 7);
    const int v_csel = (lane >> 3) & 1;
    const int sw = lane & 7;

    for (int it = 0; it < n_tiles; ++it) {
        const int st = it % kStages;
        if (!mbar_wait(&sm.full[st], (it / kStages) & 1, p.status)) return;
        const StageMeta mt = sm.meta[st];
        if (it == 0 && tid == 0) SEER_STAMP(5);
        if (mt.unit != cur_unit) {
            cur_unit = mt.unit;
            if (cur_unit == pre_unit) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) { bq[ks][0] = bq_pre[ks][0]; bq[ks][1] = bq_pre[ks][1]; }
            } else {
                load_q(bq, cur_unit);
            }
            pre_unit = cur_unit + 1;    // units follow one another (empty ones excepted)
            if (pre_unit < U) load_q(bq_pre, pre_unit);
#pragma unroll
            for (int a = 0; a < 8; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) o[a][b] = 0.f;
            m_run[0] = m_run[1] = -INFINITY;
            l_run[0] = l_run[1] = 0.f;
        }
        const int nvalid = mt.nvalid;
        if (nvalid > 16 * w) {
            const uint32_t kbase = smem_u32(sm.stage[st]);
            const uint32_t vbase = kbase + kTileBytes;
            if (nvalid < 16 * w + 16) {
                // ragged tail: rows past the sequence end may hold anything; clear this warp's
                // V rows so that 0-probability times garbage cannot produce NaN
                unsigned char* vt = sm.stage[st] + kTileBytes;
                for (int x = lane; x < 16 * 32; x += 32) {
                    int r = 16 * w + (x >> 5), part = x & 31;      // 32 x 8-byte pieces per row
                    if (r >= nvalid) {
                        int half = part >> 4, off = (part & 15) * 8;
                        *reinterpret_cast<uint2*>(vt + half * kHalfTileBytes + r * 128 + off) =
                            make_uint2(0u, 0u);
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
            }
            // ---- S^T = K . Q^T (two independent accumulator chains) ----
            float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                uint32_t a[4];
                const int c8 = ((2 * ks) & 7) + k_csel;
                ldmatrix_x4(a, kbase + (ks >> 2) * kHalfTileBytes + k_row * 128 + ((c8 ^ sw) << 4));
                if (ks & 1) mma_bf16_16816(sb, a, bq[ks][0], bq[ks][1]);
                else        mma_bf16_16816(sa, a, bq[ks][0], bq[ks][1]);
            }
            float s[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) s[x] = (sa[x] + sb[x]) * p.scale_log2;
            const int r0 = 16 * w + rw;
            if (r0 >= nvalid) s[0] = s[1] = -INFINITY;
            if (r0 + 8 >= nvalid) s[2] = s[3] = -INFINITY;
            // ---- online softmax over this warp's 16 tokens, per head column ----
            float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
            }
            const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);   // finite: >= 1 valid row
            const float al0 = fast_exp2(m_run[0] - mn0), al1 = fast_exp2(m_run[1] - mn1);
            m_run[0] = mn0; m_run[1] = mn1;
            const float p0 = fast_exp2(s[0] - mn0), p1 = fast_exp2(s[1] - mn1);
            const float p2 = fast_exp2(s[2] - mn0), p3 = fast_exp2(s[3] - mn1);
            l_run[0] = l_run[0] * al0 + (p0 + p2);
            l_run[1] = l_run[1] * al1 + (p1 + p3);
#pragma unroll
            for (int a = 0; a < 8; ++a) {
                o[a][0] *= al0; o[a][1] *= al1; o[a][2] *= al0; o[a][3] *= al1;
            }
            const uint32_t pb0 = movmatrix_trans(pack_bf16x2(p0, p1));   // tokens 0-7 of the slice
            const uint32_t pb1 = movmatrix_trans(pack_bf16x2(p2, p3));   // tokens 8-15
            // ---- O^T += V^T . P^T ----
#pragma unroll
            for (int a = 0; a < 8; ++a) {
                uint32_t f[4];
                const int c8 = ((2 * a) & 7) + v_csel;
                ldmatrix_x4_trans(f, vbase + (a >> 2) * kHalfTileBytes + v_row * 128 + ((c8 ^ sw) << 4));
                mma_bf16_16816(o[a], f, pb0, pb1);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.empty[st]);

        if (it == n_tiles - 1 && tid == 0) SEER_STAMP(6);
        if (mt.last) {
            // ---------------- end of this CTA's piece of the unit ----------------------
            float l0 = l_run[0], l1 = l_run[1];
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                l0 += __shfl_xor_sync(0xffffffffu, l0, off);
                l1 += __shfl_xor_sync(0xffffffffu, l1, off);
            }
            if (rw == 0) {
                sm.merge_ml[seg & 1][w][0][2 * qd] = m_run[0];
                sm.merge_ml[seg & 1][w][0][2 * qd + 1] = m_run[1];
                sm.merge_ml[seg & 1][w][1][2 * qd] = l0;
                sm.merge_ml[seg & 1][w][1][2 * qd + 1] = l1;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.merge_bar[0]);
            if (!mbar_wait(&sm.merge_bar[0], seg & 1, p.status)) return;
            float m_all[2], l_all[2], sc[2];
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                const int hh = 2 * qd + x;
                float mm = -INFINITY;
#pragma unroll
                for (int ww = 0; ww < kConsumerWarps; ++ww) mm = fmaxf(mm, sm.merge_ml[seg & 1][ww][0][hh]);
                float ll = 0.f;
#pragma unroll
                for (int ww = 0; ww < kConsumerWarps; ++ww) {
                    const float mw = sm.merge_ml[seg & 1][ww][0][hh];
                    ll += (mw == -INFINITY) ? 0.f : sm.merge_ml[seg & 1][ww][1][hh] * fast_exp2(mw - mm);
                }
                m_all[x] = mm;
                l_all[x] = ll;
                sc[x] = (m_run[x] == -INFINITY) ? 0.f : fast_exp2(m_run[x] - mm);
            }
            if (w > 0) {
#pragma unroll
                for (int a = 0; a < 8; ++a) {
                    const int d0 = 16 * a + rw;
                    sm.merge_o[w - 1][2 * qd][d0] = o[a][0] * sc[0];
                    sm.merge_o[w - 1][2 * qd + 1][d0] = o[a][1] * sc[1];
                    sm.merge_o[w - 1][2 * qd][d0 + 8] = o[a][2] * sc[0];
                    sm.merge_o[w - 1][2 * qd + 1][d0 + 8] = o[a][3] * sc[1];
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.merge_bar[1]);
            if (w == 0) {
                if (!mbar_wait(&sm.merge_bar[1], seg & 1, p.status)) return;
#pragma unroll
                for (int a = 0; a < 8; ++a) {
                    const int d0 = 16 * a + rw;
                    o[a][0] *= sc[0]; o[a][1] *= sc[1]; o[a][2] *= sc[0]; o[a][3] *= sc[1];
#pragma unroll
                    for (int ww = 0; ww < kConsumerWarps - 1; ++ww) {
                        o[a][0] += sm.merge_o[ww][2 * qd][d0];
                        o[a][1] += sm.merge_o[ww][2 * qd + 1][d0];
                        o[a][2] += sm.merge_o[ww][2 * qd][d0 + 8];
                        o[a][3] += sm.merge_o[ww][2 * qd + 1][d0 + 8];
                    }
                }
                const int u = mt.unit;
                const long long first = mt.unit_first;
                const int c_first = cta_of(first, T, G);
                const int c_last = cta_of(first + mt.unit_tiles - 1, T, G);
                const int n_parts = c_last - c_first + 1;
                bool write_final = (n_parts == 1);
                if (!write_final) {
                    const size_t slot = (size_t)cta + u;
                    float* po = p.part_o + slot * (kMaxGroup * kHeadDim);
#pragma unroll
                    for (int a = 0; a < 8; ++a) {
                        const int d0 = 16 * a + rw;
                        po[(2 * qd) * kHeadDim + d0] = o[a][0];
                        po[(2 * qd + 1) * kHeadDim + d0] = o[a][1];
                        po[(2 * qd) * kHeadDim + d0 + 8] = o[a][2];
                        po[(2 * qd + 1) * kHeadDim + d0 + 8] = o[a][3];
                    }
                    if (rw == 0) {
                        float* pm = p.part_ml + slot * (2 * kMaxGroup);
                        pm[2 * qd] = m_all[0];
                        pm[2 * qd + 1] = m_all[1];
                        pm[kMaxGroup + 2 * qd] = l_all[0];
                        pm[kMaxGroup + 2 * qd + 1] = l_all[1];
                    }
                    __threadfence();
                    __syncwarp();
                    int ticket = 0;
                    if (lane == 0) ticket = atomicAdd(&p.tickets[u], 1);
                    ticket = __shfl_sync(0xffffffffu, ticket, 0);
                    if (ticket == n_parts - 1) {
                        // Last piece in: log-sum-exp combine of all pieces of the unit.  Lane t takes
                        // head t/4, channels 32*(t%4) .. +31 of every piece; the loads of a pass do
                        // not depend on one another, so they are all in flight together.
                        __threadfence();
                        const int hh = lane >> 2, d0 = 32 * (lane & 3);
                        const size_t s_first = (size_t)c_first + u;
                        float M = -INFINITY;
#pragma unroll 8
                        for (int s2 = 0; s2 < n_parts; ++s2)
                            M = fmaxf(M, __ldcg(p.part_ml + (s_first + s2) * (2 * kMaxGroup) + hh));
                        float acc[32];
#pragma unroll
                        for (int x = 0; x < 32; ++x) acc[x] = 0.f;
                        float lsum = 0.f;
#pragma unroll 2
                        for (int s2 = 0; s2 < n_parts; ++s2) {
                            const float* pm = p.part_ml + (s_first + s2) * (2 * kMaxGroup);
                            const float4* qo = reinterpret_cast<const float4*>(
                                p.part_o + (s_first + s2) * (kMaxGroup * kHeadDim) + hh * kHeadDim + d0);
                            const float ms = __ldcg(pm + hh);
                            const float f = (ms == -INFINITY) ? 0.f : fast_exp2(ms - M);
                            lsum += f * __ldcg(pm + kMaxGroup + hh);
#pragma unroll
                            for (int x = 0; x < 8; ++x) {
                                const float4 v4 = __ldcg(qo + x);
                                acc[4 * x] += f * v4.x; acc[4 * x + 1] += f * v4.y;
                                acc[4 * x + 2] += f * v4.z; acc[4 * x + 3] += f * v4.w;
                            }
                        }
                        if (lane == 0) p.tickets[u] = 0;     // ready for the next launch
                        if (hh < p.group) {
                            const int i = u / p.num_kv_heads, h = u % p.num_kv_heads;
                            const size_t row = (size_t)i * p.num_q_heads + (size_t)h * p.group + hh;
                            const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
                            uint4* dst = reinterpret_cast<uint4*>(p.out + row * kHeadDim + d0);
#pragma unroll
                            for (int x = 0; x < 4; ++x) {
                                uint4 pk;
                                pk.x = pack_bf16x2(acc[8 * x] * inv, acc[8 * x + 1] * inv);
                                pk.y = pack_bf16x2(acc[8 * x + 2] * inv, acc[8 * x + 3] * inv);
                                pk.z = pack_bf16x2(acc[8 * x + 4] * inv, acc[8 * x + 5] * inv);
                                pk.w = pack_bf16x2(acc[8 * x + 6] * inv, acc[8 * x + 7] * inv);
                                dst[x] = pk;
                            }
                            if (p.lse && (lane & 3) == 0)
                                p.lse[row] = lsum > 0.f ? (M + log2f(lsum)) * 0.6931471805599453f : -INFINITY;
                        }
                    }
                }
                if (write_final) {
                    const int i = u / p.num_kv_heads, h = u % p.num_kv_heads;
                    const float inv0 = l_all[0] > 0.f ? 1.f / l_all[0] : 0.f;
                    const float inv1 = l_all[1] > 0.f ? 1.f / l_all[1] : 0.f;
                    const size_t row0 = (size_t)i * p.num_q_heads + (size_t)h * p.group + 2 * qd;
                    __nv_bfloat16* o0 = p.out + row0 * kHeadDim;
                    __nv_bfloat16* o1 = o0 + kHeadDim;
                    const bool h0 = 2 * qd < p.group, h1 = 2 * qd + 1 < p.group;
#pragma unroll
                    for (int a = 0; a < 8; ++a) {
                        const int d0 = 16 * a + rw;
                        if (h0) {
                            o0[d0] = __float2bfloat16(o[a][0] * inv0);
                            o0[d0 + 8] = __float2bfloat16(o[a][2] * inv0);
                        }
                        if (h1) {
                            o1[d0] = __float2bfloat16(o[a][1] * inv1);
                            o1[d0 + 8] = __float2bfloat16(o[a][3] * inv1);
                        }
                    }
                    if (p.lse && rw == 0) {
                        const float ln2 = 0.6931471805599453f;
                        if (h0) p.lse[row0] = l_all[0] > 0.f ? (m_all[0] + log2f(l_all[0])) * ln2 : -INFINITY;
                        if (h1) p.lse[row0 + 1] = l_all[1] > 0.f ? (m_all[1] + log2f(l_all[1])) * ln2 : -INFINITY;
                    }
                }
            }
            ++seg;
            cur_unit = -1;      // a later piece (another unit) starts from fresh state
        }
    }
    if (tid == 0) SEER_STAMP(7);
}

size_t decode_smem_bytes() { return sizeof(Smem) + 1024; }

template <bool SPARSE, bool PAGED>
cudaError_t configure() {
    return cudaFuncSetAttribute(decode_kernel<SPARSE, PAGED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)decode_smem_bytes());
}

template <bool SPARSE, bool PAGED>
int occupancy() {
    static int cached = -1;
    if (cached < 0) {
        if (configure<SPARSE, PAGED>() != cudaSuccess) return 0;
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_kernel<SPARSE, PAGED>, kThreads,
                                                          decode_smem_bytes()) != cudaSuccess)
            return 0;
        cached = n;
    }
    return cached;
}

template <bool SPARSE, bool PAGED>
cudaError_t launch(const CUtensorMap& mk, const CUtensorMap& mv, const DecodeParams& p, int grid,
                   cudaStream_t stream) {
    if (occupancy<SPARSE, PAGED>() <= 0) return cudaErrorInvalidConfiguration;
    // launched as a programmatic dependent: barrier set-up and tensor-map prefetch may overlap
    // the tail of the previous kernel in the stream (the kernel waits before its first read)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = decode_smem_bytes();
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, decode_kernel<SPARSE, PAGED>, mk, mv, p);
}

}  // namespace

int decode_ctas_per_sm(bool sparse, bool paged) {
    if (sparse) return paged ? occupancy<true, true>() : occupancy<true, false>();
    return paged ? occupancy<false, true>() : occupancy<false, false>();
}

cudaError_t launch_decode(bool sparse, bool paged, const CUtensorMap& map_k, const CUtensorMap& map_v,
                          const DecodeParams& p, int grid, cudaStream_t stream) {
    if (sparse) return paged ? launch<true, true>(map_k, map_v, p, grid, stream)
                             : launch<true, false>(map_k, map_v, p, grid, stream);
    return paged ? launch<false, true>(map_k, map_v, p, grid, stream)
                 : launch<false, false>(map_k, map_v, p, grid, stream);
}

}  // namespace seer
