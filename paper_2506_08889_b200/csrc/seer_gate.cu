// AttnGate at decode time (Eq. 1a, 1c; Sec. 3.1, 3.2).  Up to 8192 compressed keys per
// (sequence, KV head) unit the whole gate is one kernel, one thread-block cluster per unit: Q-branch
// projection + RoPE spread over the cluster's warps, block scores of each CTA's slice of the K
// compression cache, and the token-budget top-k (forced last block) by the cluster's first CTA, with
// distributed shared memory carrying the gate query and the scores between the steps.  Beyond that
// size the same steps run as a projection kernel and a score + selection kernel (the second a
// programmatic dependent of the first) that go through global memory and per-unit tickets.
#include <cstdlib>
#include <cooperative_groups.h>

#include "seer_device.cuh"
#include "seer_internal.h"

namespace cg = cooperative_groups;

namespace seer {

namespace {

constexpr int kGateThreads = 512;
constexpr int kMaxQLen = 8;                 // query tokens per sequence the gate takes
constexpr int kProjThreads = 256;

__device__ __forceinline__ float dot8(const uint4& a, const float* x) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&a);
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        float2 f = bf16x2_to_float2(h[k]);
        acc = fmaf(f.x, x[2 * k], acc);
        acc = fmaf(f.y, x[2 * k + 1], acc);
    }
    return acc;
}
__device__ __forceinline__ float dot8(const uint4& a, const uint4& b) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* g = reinterpret_cast<const __nv_bfloat162*>(&b);
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 f = bf16x2_to_float2(h[k]), e = bf16x2_to_float2(g[k]);
        acc = fmaf(f.x, e.x, acc);
        acc = fmaf(f.y, e.y, acc);
    }
    return acc;
}

// v[k], k = 0..7, summed over a group of `group` = 8, 16 or 32 neighbouring lanes, eight sums for
// 8 + (log2(group) - 3) shuffles: lanes exchange half of what they carry and go on with the other half,
// so a lane ends with the group's sum of v[r], r = its low three lane bits in reverse order.
__device__ __forceinline__ float reduce8(const float (&v)[8], int lane, int group) {
    const bool b0 = lane & 1, b1 = lane & 2, b2 = lane & 4;
    float w4[4], w2[2];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float keep = b0 ? v[i + 4] : v[i], send = b0 ? v[i] : v[i + 4];
        w4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 1);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const float keep = b1 ? w4[i + 2] : w4[i], send = b1 ? w4[i] : w4[i + 2];
        w2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
    }
    const float keep = b2 ? w2[1] : w2[0], send = b2 ? w2[0] : w2[1];
    float x = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    for (int off = 8; off < group; off <<= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
}

// Order-preserving key: larger score <-> larger key; -0 == +0; NaN below everything.
__device__ __forceinline__ uint32_t score_key(float s) {
    if (s != s) return 0u;
    uint32_t b = __float_as_uint(s);
    if (b == 0x80000000u) b = 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Split cluster barrier (all threads of all CTAs of the cluster execute both halves).
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

constexpr int kUnitThreads = 1024;          // most threads a CTA that runs the selection may have

// Inverse of score_key (NaN came out as key 0 and goes back as -inf).
__device__ __forceinline__ float key_score(uint32_t key) {
    if (key == 0u) return -INFINITY;
    return __uint_as_float((key & 0x80000000u) ? (key ^ 0x80000000u) : ~key);
}

constexpr int kSelBits = 11;                // digit width of a selection pass
constexpr int kSelBins = 1 << kSelBits;

struct SelectSmem {
    int hist[3][kSelBins];                  // one histogram per pass (at most ceil(32 / 11) passes)
    unsigned long long warp_tot[kUnitThreads / 32];
    uint32_t warp_min[kUnitThreads / 32], warp_max[kUnitThreads / 32];
    float red[kUnitThreads / 32];           // block reductions of the threshold method (its own array: the
                                            // selection that follows writes warp_min while slower warps still read)
    uint32_t pre_min, pre_max;              // smallest and largest key, when the scoring warps have found them (cluster kernel)
    uint32_t prefix;
    int rem;
    int bin_cnt;                            // one-pass path: candidates in the boundary bin ...
    int list_n;                             // ... how many of them have been listed ...
    uint32_t list[32];                      // ... and their keys
};

// Token-budget selection for one unit, run by a whole CTA.  Thread t owns the candidates
// [t*E, (t+1)*E).  A radix select (passes of 11 bits over order-preserving keys) finds the key
// of the (k-1)-th best candidate; one ordered pass then emits, in ascending block order, every
// candidate above it and the first few equal to it (the lower block number wins a tie), and
// the forced last block closes the list.  Comparisons only: the result is exact.
// NT = threads of the CTA; SMEM = the scores are in shared memory (else read from L2).
// L_known >= 0: the sequence length, already loaded.  pre: sm.pre_min / sm.pre_max hold the candidates' smallest and
// largest key and the histograms are clear (the cluster kernel sees to both before its last cluster barrier).
template <int NT, bool CACHED, bool SMEM>
__device__ void select_unit(const GateParams& p, int u, const float* sc, SelectSmem& sm, int L_known = -1, bool pre = false) {
    constexpr int kCachedT = CACHED ? (NT >= 1024 ? 4 : 8) : 1;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int i = u / p.num_kv_heads;
    int32_t* dst = p.block_idx + (size_t)u * p.max_sel;
    const int L = L_known >= 0 ? L_known : p.seq_lens[i];
    const int n_i = L > 0 ? (L + p.block_size - 1) / p.block_size : 0;
    if (n_i <= 0) {
        for (int e = tid; e < p.max_sel; e += NT) dst[e] = -1;
        if (tid == 0) p.block_cnt[u] = 0;
        return;
    }
    int k = max(p.token_budget / p.block_size, 1);
    k = min(k, min(n_i, p.max_sel));
    // The blocks that hold a query token's own position, j_f .. n_i - 1, are always taken (one block,
    // the last, for a single query token); the candidates are the blocks before them.
    const int j_f = max(0, L - p.q_len) / p.block_size;
    const int n_forced = min(n_i - j_f, p.max_sel);
    const int n_cand = min(j_f, p.max_blocks);
    int need = max(0, min(k - n_forced, n_cand));    // candidates to take besides the forced blocks
    const int E = (n_cand + NT - 1) / NT;
    const int j_lo = min(n_cand, tid * E), j_hi = min(n_cand, j_lo + E);

    auto score_at = [&](int j) -> float { return SMEM ? sc[j] : __ldcg(sc + j); };
    uint32_t keys[kCachedT];
    if (CACHED) {
#pragma unroll
        for (int e = 0; e < kCachedT; ++e) keys[e] = (j_lo + e < j_hi) ? score_key(score_at(j_lo + e)) : 0u;
    }
    auto key_at = [&](int e) -> uint32_t { return score_key(score_at(j_lo + e)); };

    if (p.threshold_mode) {
        // Threshold method (Sec. 3.1): softmax of the scores over the candidate blocks; the blocks
        // with probability above tau are taken.  They are the `above` highest-scoring candidates
        // (equal scores have equal probabilities), so only the count differs from the budget method.
        auto block_reduce = [&](float v, bool is_max) -> float {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const float o = __shfl_xor_sync(0xffffffffu, v, off);
                v = is_max ? fmaxf(v, o) : v + o;
            }
            __syncthreads();                                   // the scratch may still be in use
            if (lane == 0) sm.red[warp] = v;
            __syncthreads();
            float r = is_max ? -INFINITY : 0.f;
#pragma unroll
            for (int w2 = 0; w2 < NT / 32; ++w2) {
                const float o = sm.red[w2];
                r = is_max ? fmaxf(r, o) : r + o;
            }
            return r;
        };
        auto for_each_score = [&](auto&& fn) {
            if (CACHED) {
#pragma unroll
                for (int e = 0; e < kCachedT; ++e)
                    if (j_lo + e < j_hi) fn(key_score(keys[e]));
            } else {
                for (int e = 0; j_lo + e < j_hi; ++e) fn(key_score(key_at(e)));
            }
        };
        float mx = -INFINITY;
        for_each_score([&](float v) { mx = fmaxf(mx, v); });
        mx = block_reduce(mx, true);
        float z = 0.f;
        for_each_score([&](float v) { z += __expf(v - mx); });
        z = block_reduce(z, false);
        float cnt_above = 0.f;
        for_each_score([&](float v) { cnt_above += (__expf(v - mx) > p.threshold * z) ? 1.f : 0.f; });
        const int above = (int)(block_reduce(cnt_above, false) + 0.5f);
        need = max(0, min(min(above, p.max_sel - n_forced), n_cand));
    }

    uint32_t thr = 0u;                               // key of the need-th best candidate
    int take_eq = n_cand;                            // candidates equal to thr that are taken
    if (need > 0 && need < n_cand) {
        // The keys of real scores crowd into a few exponent values, so digits of the raw key make
        // for a handful of hot histogram bins.  The passes therefore work on key - min(key), whose
        // significant bits (those of max - min) are spread evenly: first the block-wide min and max.
        uint32_t kmin = 0xffffffffu, kmax = 0u;
        if (pre) {
            kmin = sm.pre_min;
            kmax = sm.pre_max;
        } else {
            if (CACHED) {
#pragma unroll
                for (int e = 0; e < kCachedT; ++e)
                    if (j_lo + e < j_hi) { kmin = min(kmin, keys[e]); kmax = max(kmax, keys[e]); }
            } else {
                for (int e = 0; j_lo + e < j_hi; ++e) { const uint32_t key = key_at(e); kmin = min(kmin, key); kmax = max(kmax, key); }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, off));
                kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, off));
            }
            if (lane == 0) { sm.warp_min[warp] = kmin; sm.warp_max[warp] = kmax; }
            for (int x = tid; x < 3 * kSelBins; x += NT) (&sm.hist[0][0])[x] = 0;
            __syncthreads();
#pragma unroll
            for (int w2 = 0; w2 < NT / 32; ++w2) { kmin = min(kmin, sm.warp_min[w2]); kmax = max(kmax, sm.warp_max[w2]); }
        }
        int bits_left = 32 - __clz(max(kmax - kmin, 1u));     // significant bits of key - kmin
        uint32_t prefix = 0u;                                  // the digits found so far, of thr - kmin
        int rem = need;
        constexpr int kBinsPerThread = kSelBins / NT;
        // One-pass path.  Scores spread over [smin, smax] like a bell curve put at most a few
        // candidates into any of 2048 equal-width bins, so one histogram over the monotone map
        //     bin(s) = floor((s - smin) * 2047 / (smax - smin))
        // leaves a boundary bin with a handful of candidates, which one warp ranks directly.  The map
        // only has to be monotone for the result to be exact (equal scores share a bin, a larger score
        // never lands in a lower one); when it is unusable (non-finite range) or the boundary bin
        // holds more than 32 candidates, the radix passes below do the job.
        if (CACHED) {
            const float smin = key_score(kmin), smax = key_score(kmax);
            const float range = smax - smin, scale = 2047.f / range;
            if (smin > -INFINITY && range > 0.f && range < INFINITY && scale < INFINITY) {
                int* hist = sm.hist[2];
                auto bin_of = [&](uint32_t key) -> int {
                    return min(kSelBins - 1, (int)((key_score(key) - smin) * scale));
                };
                int my_bin[kCachedT];
#pragma unroll
                for (int e = 0; e < kCachedT; ++e) {
                    my_bin[e] = -1;
                    if (j_lo + e < j_hi) { my_bin[e] = bin_of(keys[e]); atomicAdd(&hist[my_bin[e]], 1); }
                }
                if (tid == 0) sm.list_n = 0;
                __syncthreads();
                int c[kBinsPerThread], mine = 0;
#pragma unroll
                for (int x = 0; x < kBinsPerThread; ++x) { c[x] = hist[kSelBins - 1 - kBinsPerThread * tid - x]; mine += c[x]; }
                int incl = mine;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += t;
                }
                if (lane == 31) sm.warp_tot[warp] = (unsigned long long)incl;
                __syncthreads();
                int above = incl - mine;
#pragma unroll
                for (int w2 = 0; w2 < NT / 32; ++w2) above += (w2 < warp) ? (int)sm.warp_tot[w2] : 0;
                if (above < rem && rem <= above + mine) {
#pragma unroll
                    for (int x = 0; x < kBinsPerThread; ++x) {
                        if (above < rem && rem <= above + c[x]) {
                            sm.prefix = (uint32_t)(kSelBins - 1 - kBinsPerThread * tid - x);
                            sm.rem = rem - above;
                            sm.bin_cnt = c[x];
                        }
                        above += c[x];
                    }
                }
                __syncthreads();
                const int bbin = (int)sm.prefix, brem = sm.rem, bcnt = sm.bin_cnt;
                if (bcnt <= 32) {
                    // list the boundary bin's keys; warp 0 finds the brem-th largest among them
#pragma unroll
                    for (int e = 0; e < kCachedT; ++e)
                        if (my_bin[e] == bbin) sm.list[atomicAdd(&sm.list_n, 1)] = keys[e];
                    __syncthreads();
                    if (warp == 0) {
                        const uint32_t mykey = lane < bcnt ? sm.list[lane] : 0u;
                        int gt = 0, ge = 0;
                        for (int m2 = 0; m2 < bcnt; ++m2) {
                            const uint32_t km = __shfl_sync(0xffffffffu, mykey, m2);
                            gt += km > mykey;
                            ge += km >= mykey;
                        }
                        if (lane < bcnt && gt < brem && brem <= ge) {     // all such lanes hold the same key
                            sm.prefix = mykey;
                            sm.rem = brem - gt;
                        }
                    }
                    __syncthreads();
                    thr = sm.prefix;
                    take_eq = sm.rem;
                    bits_left = 0;                         // the radix passes are not needed
                } else {
                    for (int x = tid; x < kSelBins; x += NT) hist[x] = 0;   // used again by the third pass
                }
            }
        }
        const bool radix = bits_left > 0;
        for (int pass = 0; bits_left > 0; ++pass) {
            const int wbits = min(kSelBits, bits_left), shift = bits_left - wbits;
            int* hist = sm.hist[pass];
            auto count = [&](uint32_t key) {
                const uint32_t rel = key - kmin;
                // 64-bit shift: shift + wbits can be 32
                if ((uint32_t)((unsigned long long)rel >> (shift + wbits)) == prefix)
                    atomicAdd(&hist[(rel >> shift) & ((1u << wbits) - 1u)], 1);
            };
            if (CACHED) {
#pragma unroll
                for (int e = 0; e < kCachedT; ++e)
                    if (j_lo + e < j_hi) count(keys[e]);
            } else {
                for (int e = 0; j_lo + e < j_hi; ++e) count(key_at(e));
            }
            __syncthreads();
            // thread t owns bins (kSelBins-1 - kBinsPerThread*t) downwards; a block scan gives the number
            // of keys in all higher bins, then the thread that straddles `rem` walks its own bins
            int c[kBinsPerThread], mine = 0;
#pragma unroll
            for (int x = 0; x < kBinsPerThread; ++x) { c[x] = hist[kSelBins - 1 - kBinsPerThread * tid - x]; mine += c[x]; }
            unsigned long long incl = (unsigned long long)mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            if (lane == 31) sm.warp_tot[warp] = incl;
            __syncthreads();
            int above = (int)incl - mine;
#pragma unroll
            for (int w2 = 0; w2 < NT / 32; ++w2) above += (w2 < warp) ? (int)sm.warp_tot[w2] : 0;
            if (above < rem && rem <= above + mine) {
#pragma unroll
                for (int x = 0; x < kBinsPerThread; ++x) {
                    if (above < rem && rem <= above + c[x]) {
                        sm.prefix = (prefix << wbits) | (uint32_t)(kSelBins - 1 - kBinsPerThread * tid - x);
                        sm.rem = rem - above;
                    }
                    above += c[x];
                }
            }
            __syncthreads();
            prefix = sm.prefix;
            rem = sm.rem;
            bits_left = shift;
        }
        if (radix) {
            thr = kmin + prefix;
            take_eq = rem;
        }
    }

    if (need > 0) {
        int n_gt = 0, n_eq = 0;
        if (CACHED) {
#pragma unroll
            for (int e = 0; e < kCachedT; ++e)
                if (j_lo + e < j_hi) { n_gt += keys[e] > thr; n_eq += keys[e] == thr; }
        } else {
            for (int e = 0; j_lo + e < j_hi; ++e) {
                const uint32_t key = key_at(e);
                n_gt += key > thr; n_eq += key == thr;
            }
        }
        // one block-wide exclusive scan of both counts packed into one 64-bit word
        const unsigned long long packed = ((unsigned long long)n_gt << 32) | (unsigned long long)n_eq;
        unsigned long long incl = packed;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) sm.warp_tot[warp] = incl;
        __syncthreads();
        unsigned long long base = 0;
#pragma unroll
        for (int w2 = 0; w2 < NT / 32; ++w2) base += (w2 < warp) ? sm.warp_tot[w2] : 0ull;
        const unsigned long long excl = base + incl - packed;
        const int gt_before = (int)(excl >> 32);
        int eq_rank = (int)(excl & 0xffffffffull);
        int pos = gt_before + min(eq_rank, take_eq);
        if (CACHED) {
#pragma unroll
            for (int e = 0; e < kCachedT; ++e) {
                if (j_lo + e < j_hi) {
                    const bool gt = keys[e] > thr, eq = keys[e] == thr;
                    if (gt || (eq && eq_rank < take_eq)) dst[pos++] = j_lo + e;
                    eq_rank += eq;
                }
            }
        } else {
            for (int e = 0; j_lo + e < j_hi; ++e) {
                const uint32_t key = key_at(e);
                const bool gt = key > thr, eq = key == thr;
                if (gt || (eq && eq_rank < take_eq)) dst[pos++] = j_lo + e;
                eq_rank += eq;
            }
        }
    }
    if (tid < n_forced) dst[need + tid] = n_i - n_forced + tid;      // the always-active last block(s)
    if (tid == 0) p.block_cnt[u] = need + n_forced;
    for (int e = need + n_forced + tid; e < p.max_sel; e += NT) dst[e] = -1;
}

template <int NT, bool SMEM>
__device__ __forceinline__ void select_dispatch(const GateParams& p, int u, const float* sc, SelectSmem& sm, int L_known = -1,
                                                bool pre = false) {
    if (p.max_blocks <= (NT >= 1024 ? 4 : 8) * NT) select_unit<NT, true, SMEM>(p, u, sc, sm, L_known, pre);
    else select_unit<NT, false, SMEM>(p, u, sc, sm, L_known, pre);
}

// The unit's list (entries, count, padding) is complete: tell a kernel that waits for it per unit.
__device__ __forceinline__ void publish_list(const GateParams& p, int u) {
    if (!p.list_flags) return;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        st_release_gpu(p.list_flags + u, p.list_gen);
    }
}

// Selection on caller-provided scores: one CTA per unit.
__global__ void __launch_bounds__(kGateThreads) gate_select_only_kernel(const GateParams p) {
    __shared__ SelectSmem sm;
    const int u = blockIdx.x;
    pdl_wait();
    pdl_launch_dependents();
    select_dispatch<kGateThreads, false>(p, u, p.scores_in + (size_t)u * p.max_blocks, sm);
    publish_list(p, u);
}

// ---- q_gate = RoPE_{L_i - 1}( W_q[h] . concat_g(Q_nope) )  (Eq. 1a) ---------------------------
// grid (B*Hkv, d_gate/32, q_len): a CTA computes 16 rotary pairs of one query token's gate query
// (q_gate [B*Hkv][q_len][d_gate]); each of its 8 warps takes two pairs,
// i.e. rows c, c+1, c+d_gate/2, c+1+d_gate/2, with all of their loads in flight together.
// NIT = 16-byte pieces of a row per lane (row length g*128 bf16 = g*16 pieces over 32 lanes).
template <int NIT>
__global__ void __launch_bounds__(kProjThreads) gate_qproj_kernel(const GateParams p) {
    pdl_wait();
    pdl_launch_dependents();      // the score kernel may start requesting its keys
    const int u = blockIdx.x, i = u / p.num_kv_heads, h = u % p.num_kv_heads;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n = p.group * kHeadDim, chunks = n / 8, half = p.d_gate / 2;
    const int c0 = blockIdx.y * 16 + warp * 2;
    if (c0 >= half) return;
    const int t = blockIdx.z;                          // query token (its position: L - q_len + t)
    const uint4* xsrc = reinterpret_cast<const uint4*>(
        p.q_nope + (((size_t)i * p.q_len + t) * p.num_q_heads + (size_t)h * p.group) * kHeadDim);
    const int L = __ldg(p.seq_lens + i);
    uint4 xv[NIT], wv[4][NIT];
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int ch = lane + 32 * it;
        xv[it] = ch < chunks ? __ldg(xsrc + ch) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int r = c0 + (k & 1) + (k >> 1) * half;
        const uint4* wrow = reinterpret_cast<const uint4*>(p.w_q + ((size_t)h * p.d_gate + r) * n);
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int ch = lane + 32 * it;
            wv[k][it] = ch < chunks ? __ldg(wrow + ch) : make_uint4(0u, 0u, 0u, 0u);
        }
    }
    float acc[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        acc[k] = 0.f;
#pragma unroll
        for (int it = 0; it < NIT; ++it) acc[k] += dot8(wv[k][it], xv[it]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], off);
    }
    if (lane < 2) {
        const int c = c0 + lane;
        float sn, cs;
        rope_sincos((double)max(L - p.q_len + t, 0), p.inv_freq[c], &sn, &cs);
        const float a = lane ? acc[1] : acc[0], b = lane ? acc[3] : acc[2];
        float* dst = p.q_gate + ((size_t)u * p.q_len + t) * p.d_gate;
        dst[c] = a * cs - b * sn;
        dst[c + half] = b * cs + a * sn;
    }
}

// ---- scores (Eq. 1c without the softmax) and selection ------------------------------------------
// grid (S, B*Hkv): the compressed keys of one (sequence, KV head) unit are cut into S slices of
// `per` entries.  A slice is one flat run of 16-byte pieces; thread t takes pieces t, t+512, ...
// (kBatch in flight at a time; the first batch is requested before the kernel waits for the
// projection kernel), and the d_gate/8 neighbouring lanes that hold one key's pieces add up by
// shuffles.  Each CTA publishes its scores and takes a ticket; the CTA that draws the unit's
// last ticket runs the selection over all of the unit's scores.  No CTA waits for another.
#ifdef SEER_GATE_TRACE
#define GATE_STAMP(k) do { if (threadIdx.x == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); \
    reinterpret_cast<unsigned long long*>(p.status)[((size_t)blockIdx.y * gridDim.x + blockIdx.x) * 16 + (k)] = t_; } } while (0)
#else
#define GATE_STAMP(k) ((void)0)
#endif

__global__ void __launch_bounds__(kGateThreads, 2) gate_score_select_kernel(const GateParams p, int per) {
    __shared__ SelectSmem sm;
    __shared__ int is_last;
    const int u = blockIdx.y, i = u / p.num_kv_heads;
    const int S = gridDim.x, slice = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31;
    const int lpk = p.d_gate / 8;                      // lanes per key: 8, 16 or 32
    const int csub = tid & (lpk - 1);
    const int j0 = min(p.max_blocks, slice * per), j1 = min(p.max_blocks, j0 + per);
    const uint4* kc = reinterpret_cast<const uint4*>(p.kcomp + ((size_t)u * p.max_blocks + j0) * p.d_gate);
    const int total = (j1 - j0) * lpk;
    constexpr int kBatch = 8;
    uint4 kv[kBatch];
#pragma unroll
    for (int k = 0; k < kBatch; ++k) {                 // entries past n_i - 1 exist in memory: harmless
        const int c = k * kGateThreads + tid;
        kv[k] = c < total ? __ldg(kc + c) : make_uint4(0u, 0u, 0u, 0u);
    }
    GATE_STAMP(0);
    pdl_wait();                                        // q_gate is complete from here on
    GATE_STAMP(1);
    pdl_launch_dependents();
    const int L = __ldg(p.seq_lens + i);
    const int q_len = p.q_len;
    // the blocks wholly before the first query token (for one token: all but the last block)
    const int n_cand = min(max(0, L - q_len) / p.block_size, p.max_blocks);
    float* sc_out = p.scores + (size_t)u * p.max_blocks;
    // this thread's 8 channels of every query token's gate query
    const float* qbase = p.q_gate + (size_t)u * q_len * p.d_gate + 8 * csub;
    float qsub[8];
    auto load_q = [&](int t) {
        const float4 a = __ldcg(reinterpret_cast<const float4*>(qbase + (size_t)t * p.d_gate));
        const float4 b = __ldcg(reinterpret_cast<const float4*>(qbase + (size_t)t * p.d_gate + 4));
        qsub[0] = a.x; qsub[1] = a.y; qsub[2] = a.z; qsub[3] = a.w;
        qsub[4] = b.x; qsub[5] = b.y; qsub[6] = b.z; qsub[7] = b.w;
    };
    load_q(0);
    const float inv = rsqrtf((float)p.d_gate);
    const int lpk_shift = 31 - __clz(lpk);
    const int krev = ((lane & 1) << 2) | (lane & 2) | ((lane >> 2) & 1);
    for (int cb = 0; cb < total; cb += kGateThreads * kBatch) {
        // a key's score is the largest of its dot products with the query tokens' gate queries; after
        // reduce8 a lane holds the sum of the key of its piece number krev
        float best = -INFINITY;
        for (int t = 0; t < q_len; ++t) {
            if (q_len > 1) load_q(t);
            float acc[kBatch];
#pragma unroll
            for (int k = 0; k < kBatch; ++k) acc[k] = dot8(kv[k], qsub);
            const float x = reduce8(acc, lane, lpk);
            best = q_len > 1 ? fmaxf(best, x) : x;
        }
        const int cb_now = cb;
        if (cb + kGateThreads * kBatch < total) {      // next batch on its way while this one is stored
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int c = cb + (kBatch + k) * kGateThreads + tid;
                kv[k] = c < total ? __ldg(kc + c) : make_uint4(0u, 0u, 0u, 0u);
            }
        }
        const int c = cb_now + krev * kGateThreads + tid;
        const int j = j0 + (c >> lpk_shift);
        if (c < total && (csub & ~7) == 0 && j < n_cand) __stcg(sc_out + j, best * inv);
    }
    // ---- ticket: the last slice of the unit to finish does the selection --------------------
    GATE_STAMP(2);
    __threadfence();
    __syncthreads();
    GATE_STAMP(3);
    if (tid == 0) {
        const int t = atomicAdd(&p.tickets[u], 1);
        is_last = (t == S - 1);
        if (is_last) p.tickets[u] = 0;               // ready for the next launch
    }
    __syncthreads();
    GATE_STAMP(4);
    if (!is_last) return;
    select_dispatch<kGateThreads, false>(p, u, sc_out, sm);   // reads the scores with ld.cg, after the ticket
    publish_list(p, u);
    GATE_STAMP(5);
}

// ---- the whole gate of one unit in one thread-block cluster -------------------------------------
// grid (S, B*Hkv) with cluster (S, 1, 1): the S CTAs of a cluster share one (sequence, KV head) unit.
//   1. Every warp of the cluster takes rotary pairs of the Q branch (rows c and c + d_gate/2 of
//      W_q[h]; the rows of its first pair are requested before the kernel waits for its
//      predecessor, W_q being a constant), applies RoPE and stores the two results into the
//      shared memory of all S CTAs (distributed shared memory).
//   2. Each CTA scores its slice of the compressed keys (requested right after the wait, so they
//      travel during step 1) and stores the scores into the shared memory of the cluster's first CTA.
//   3. The first CTA runs the selection on the scores in its shared memory.
// Between the steps the cluster meets at its hardware barrier; nothing goes through global memory
// and nobody takes tickets.  NIT = 16-byte pieces of a W_q row per lane.
template <int NIT, bool MULTI>
__global__ void __launch_bounds__(kGateThreads, 2) gate_cluster_kernel(const GateParams p, int per) {
    extern __shared__ __align__(16) float sc_all[];    // scores [max_blocks] (used in the first CTA), staged keys
    __shared__ float qg[MULTI ? kMaxQLen : 1][kMaxDGate];   // gate queries of the unit's query tokens
    const int q_len = MULTI ? p.q_len : 1;             // (a compile-time 1 for plain decoding)
    __shared__ SelectSmem sm;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = (int)cluster.num_blocks(), slice = (int)cluster.block_rank();
    const int u = blockIdx.y, i = u / p.num_kv_heads, h = u % p.num_kv_heads;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = p.group * kHeadDim, chunks = n / 8, half = p.d_gate / 2;
    const int gw = slice * (kGateThreads / 32) + warp, n_gw = S * (kGateThreads / 32);
    // Another CTA's shared memory may only be written once that CTA is known to be running: every
    // CTA signals its start here and waits for the others just before step 1's remote stores.
    cluster_arrive();
    // Work items of the projection: (query token t, rotary pair c), item = t * half + c, dealt to the
    // cluster's warps round robin.  W_q rows of this warp's first item: constants, requested before the wait.
    const int n_items = q_len * half;
    uint4 wv[2][NIT];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const uint4* wrow = reinterpret_cast<const uint4*>(p.w_q + ((size_t)h * p.d_gate + gw % half + k * half) * n);
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int ch = lane + 32 * it;
            wv[k][it] = (gw < n_items && ch < chunks) ? __ldg(wrow + ch) : make_uint4(0u, 0u, 0u, 0u);
        }
    }
    // The slice's compressed keys are asked into L2 meanwhile (a hint only; they are read after the
    // wait): entries of complete earlier blocks do not change any more, so in a decode step the
    // key stream overlaps the predecessor kernel.
    {
        const int pj0 = min(p.max_blocks, slice * per), pj1 = min(p.max_blocks, pj0 + per);
        const char* base = reinterpret_cast<const char*>(p.kcomp + ((size_t)u * p.max_blocks + pj0) * p.d_gate);
        const int bytes = (pj1 - pj0) * p.d_gate * 2;
        for (int off = tid * 512; off < bytes; off += kGateThreads * 512) prefetch_l2(base + off, min(512, bytes - off));
    }
    GATE_STAMP(0);
    pdl_wait();                                        // queries, lengths and compressed keys are final
    GATE_STAMP(1);
    pdl_launch_dependents();
    // This slice's keys: one flat run of 16-byte pieces, thread t taking pieces t, t + 512, ...
    // The first kBatch pieces per thread go straight into shared memory by asynchronous copies, issued
    // now, so that they travel during the projection; the next kBatch are requested into registers
    // once the projection has freed them; any further ones follow in register batches.
    const int lpk = p.d_gate / 8;                      // lanes per key: 8, 16 or 32
    const int csub = tid & (lpk - 1);
    const int j0 = min(p.max_blocks, slice * per), j1 = min(p.max_blocks, j0 + per);
    const uint4* kc = reinterpret_cast<const uint4*>(p.kcomp + ((size_t)u * p.max_blocks + j0) * p.d_gate);
    const int total = (j1 - j0) * lpk;
    constexpr int kBatch = 8;
    uint4* staged = reinterpret_cast<uint4*>(sc_all + ((p.max_blocks + 3) & ~3));     // [kBatch * 512] pieces
    // The small loads the projection waits for -- the sequence length and the pre-RoPE queries of this
    // warp's first work item -- are requested before the keys: behind 128 KB of key requests they would
    // come back microseconds later.
    const int L = __ldg(p.seq_lens + i);
    uint4 xv0[NIT];
    {
        const int t0 = gw / half;
        const uint4* xsrc = reinterpret_cast<const uint4*>(
            p.q_nope + (((size_t)i * q_len + min(t0, q_len - 1)) * p.num_q_heads + (size_t)h * p.group) * kHeadDim);
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int ch = lane + 32 * it;
            xv0[it] = ch < chunks ? __ldg(xsrc + ch) : make_uint4(0u, 0u, 0u, 0u);
        }
    }
#pragma unroll
    for (int k = 0; k < kBatch; ++k) {                 // entries past n_i - 1 exist in memory: harmless
        const int pc = k * kGateThreads + tid;
        if (pc < total) cp_async16(staged + pc, kc + pc);
    }
    // The first CTA, which will select, clears its histograms and the two words the scoring warps fold
    // the smallest and largest key into (remote atomics, after the first cluster barrier) now, while
    // the keys travel: the selection then starts with both in hand.
    if (slice == 0) {
        for (int x = tid; x < 3 * kSelBins; x += kGateThreads) (&sm.hist[0][0])[x] = 0;
        if (tid == 0) { sm.pre_min = 0xffffffffu; sm.pre_max = 0u; }
    }
    cluster_wait();                                    // every CTA of the cluster has started
    // ---- 1. gate queries --------------------------------------------------------------------------
    for (int item = gw; item < n_items; item += n_gw) {
        const int t = item / half, c = item - t * half;
        const uint4* xsrc = reinterpret_cast<const uint4*>(
            p.q_nope + (((size_t)i * q_len + t) * p.num_q_heads + (size_t)h * p.group) * kHeadDim);
        uint4 xv[NIT];
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int ch = lane + 32 * it;
            xv[it] = item == gw ? xv0[it] : (ch < chunks ? __ldg(xsrc + ch) : make_uint4(0u, 0u, 0u, 0u));
        }
        if (item != gw) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const uint4* wrow = reinterpret_cast<const uint4*>(p.w_q + ((size_t)h * p.d_gate + c + k * half) * n);
#pragma unroll
                for (int it = 0; it < NIT; ++it) {
                    const int ch = lane + 32 * it;
                    wv[k][it] = ch < chunks ? __ldg(wrow + ch) : make_uint4(0u, 0u, 0u, 0u);
                }
            }
        }
        float a = 0.f, b = 0.f;
#pragma unroll
        for (int it = 0; it < NIT; ++it) { a += dot8(wv[0][it], xv[it]); b += dot8(wv[1][it], xv[it]); }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            a += __shfl_xor_sync(0xffffffffu, a, off);
            b += __shfl_xor_sync(0xffffffffu, b, off);
        }
        // query token t sits at position L - q_len + t
        float sn, cs;
        rope_sincos((double)max(L - q_len + t, 0), p.inv_freq[c], &sn, &cs);
        const float ra = a * cs - b * sn, rb = b * cs + a * sn;
        if (lane < S) {                                // lane r stores into CTA r of the cluster
            float* dst = cluster.map_shared_rank(&qg[0][0], lane) + t * kMaxDGate;
            dst[c] = ra;
            dst[c + half] = rb;
        }
    }
    // second batch of keys, into the registers that held W_q and the queries
    uint4 kv[kBatch];
#pragma unroll
    for (int k = 0; k < kBatch; ++k) {
        const int pc = (kBatch + k) * kGateThreads + tid;
        kv[k] = pc < total ? __ldg(kc + pc) : make_uint4(0u, 0u, 0u, 0u);
    }
    GATE_STAMP(2);
    cluster.sync();
    GATE_STAMP(3);
    // ---- 2. scores of this slice, into the first CTA's shared memory ---------------------------
    const int n_cand = min(max(0, L - q_len) / p.block_size, p.max_blocks);   // blocks before the query tokens' own
    float* sc0 = cluster.map_shared_rank(sc_all, 0);
    float* sc_user = p.scores_user ? p.scores_user + (size_t)u * p.max_blocks : nullptr;
    const float inv = rsqrtf((float)p.d_gate);
    // A key's score is the largest of its dot products with the query tokens' gate queries.  A thread holds
    // one piece of each of kBatch = 8 keys, the lpk lanes of a group the same 8 keys; reduce8 adds up over the
    // group so that every lane ends with the sum of ONE of the keys (of piece number krev, the lane's low
    // three bits reversed): each exchange halves the values a lane carries on.  Lanes 0..7 of a group store.
    const int lpk_shift = 31 - __clz(lpk);
    const int krev = ((lane & 1) << 2) | (lane & 2) | ((lane >> 2) & 1);
    const bool storer = (csub & ~7) == 0;
    uint32_t kmn = 0xffffffffu, kmx = 0u;              // smallest and largest key among the scores this thread stores
    auto score_batch = [&](auto&& piece, int cb) {
        float best = -INFINITY;
        for (int t = 0; t < q_len; ++t) {
            float qsub[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) qsub[c] = qg[t][8 * csub + c];
            float acc[kBatch];
#pragma unroll
            for (int k = 0; k < kBatch; ++k) acc[k] = dot8(piece(k), qsub);
            const float x = reduce8(acc, lane, lpk);
            best = MULTI ? fmaxf(best, x) : x;
        }
        const int j = j0 + ((cb + krev * kGateThreads + tid) >> lpk_shift);
        if (storer && j < j1 && j < n_cand) {
            const float v = best * inv;
            sc0[j] = v;
            if (sc_user) sc_user[j] = v;
            const uint32_t key = score_key(v);
            kmn = min(kmn, key);
            kmx = max(kmx, key);
        }
    };
    // Batches alternate between the staged area (each thread reads back the pieces it copied itself)
    // and the registers; while one is scored the one after the next is on its way into the place
    // that has just been freed.
    constexpr int kPieces = kGateThreads * kBatch;
    for (int cb = 0;;) {
        cp_async_wait_all();
        if (cb == 0) GATE_STAMP(8);
        score_batch([&](int k) { const int pc = cb + k * kGateThreads + tid; return pc < total ? staged[pc - cb] : make_uint4(0u, 0u, 0u, 0u); }, cb);
        if (cb == 0) GATE_STAMP(9);
        cb += kPieces;
        if (cb >= total) break;
        if (cb + kPieces < total) {
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int pc = cb + kPieces + k * kGateThreads + tid;
                if (pc < total) cp_async16(staged + (pc - cb - kPieces), kc + pc);
            }
        }
        score_batch([&](int k) { return kv[k]; }, cb);
        cb += kPieces;
        if (cb >= total) break;
        if (cb + kPieces < total) {
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int pc = cb + kPieces + k * kGateThreads + tid;
                kv[k] = pc < total ? __ldg(kc + pc) : make_uint4(0u, 0u, 0u, 0u);
            }
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        kmn = min(kmn, __shfl_xor_sync(0xffffffffu, kmn, off));
        kmx = max(kmx, __shfl_xor_sync(0xffffffffu, kmx, off));
    }
    if (lane == 0 && kmn <= kmx) {
        atomicMin(cluster.map_shared_rank(&sm.pre_min, 0), kmn);
        atomicMax(cluster.map_shared_rank(&sm.pre_max, 0), kmx);
    }
    GATE_STAMP(4);
    cluster.sync();
    GATE_STAMP(5);
    // ---- 3. selection by the first CTA ----------------------------------------------------------
    if (slice != 0) return;
    select_dispatch<kGateThreads, true>(p, u, sc_all, sm, L, true);
    publish_list(p, u);
    GATE_STAMP(6);
}

constexpr int kClusterStageBytes = 8 * kGateThreads * 16;   // the staged first batch of a slice's keys
constexpr int kClusterMaxBlocks = 8192;     // compressed keys per unit the cluster kernel holds in shared memory

template <int NIT, bool MULTI>
cudaError_t launch_gate_cluster(const GateParams& p, int S, int per, cudaStream_t stream) {
    static bool configured[kMaxDevices] = {};
    const int slot = current_device_slot();
    if (!configured[slot]) {
        const cudaError_t e = cudaFuncSetAttribute(gate_cluster_kernel<NIT, MULTI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   kClusterMaxBlocks * (int)sizeof(float) + kClusterStageBytes);
        if (e != cudaSuccess) return e;
        configured[slot] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S, p.batch * p.num_kv_heads);
    cfg.blockDim = dim3(kGateThreads);
    cfg.dynamicSmemBytes = (size_t)((p.max_blocks + 3) & ~3) * sizeof(float) + kClusterStageBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = S;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gate_cluster_kernel<NIT, MULTI>, p, per);
}

}  // namespace

bool gate_one_kernel(int max_blocks) { return max_blocks <= kClusterMaxBlocks; }

cudaError_t launch_gate_select(const GateParams& p, cudaStream_t stream, int* launched) {
    const int U = p.batch * p.num_kv_heads;
    *launched = 0;
    if (p.scores_in) {
        *launched = 1;
        return launch_pdl(gate_select_only_kernel, dim3(U), dim3(kGateThreads), 0, stream, p);
    }
    const int nit = (p.group * kHeadDim / 8 + 31) / 32;
    cudaError_t e;
    if (p.max_blocks <= kClusterMaxBlocks) {
        // one cluster per unit: slices of about 512 compressed keys, at most 8 CTAs
        int S = (p.max_blocks + 511) / 512;
        S = S < 1 ? 1 : (S > 8 ? 8 : S);
        // With few units (small batches) the clusters are widened while they all still fit the SMs at two CTAs
        // each (what the kernel's shared memory allows) and a slice keeps 128 keys or more: the projection's rows and the keys of a unit are then spread
        // over more SMs, and the chain of phases gets shorter.
        {
            static int sm_count[kMaxDevices] = {};
            const int slot = current_device_slot();
            if (sm_count[slot] == 0) {
                int dev = 0, n = 0;
                if (cudaGetDevice(&dev) == cudaSuccess &&
                    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
                    sm_count[slot] = n;
                else
                    sm_count[slot] = 1;
            }
            static int widen = -1;
            if (widen < 0) {
                const char* e = getenv("SEER_GATE_WIDEN");
                widen = e ? atoi(e) : 2;         // (CTAs per SM that the clusters may fill; 0: no widening)
            }
            while (widen && 2 * S <= 8 && U * 2 * S <= widen * sm_count[slot] && (p.max_blocks + 2 * S - 1) / (2 * S) >= 128) S *= 2;
        }
        const int per = (p.max_blocks + S - 1) / S;
        const bool multi = p.q_len > 1;
        switch (nit) {
            case 1: e = multi ? launch_gate_cluster<1, true>(p, S, per, stream) : launch_gate_cluster<1, false>(p, S, per, stream); break;
            case 2: e = multi ? launch_gate_cluster<2, true>(p, S, per, stream) : launch_gate_cluster<2, false>(p, S, per, stream); break;
            case 3: e = multi ? launch_gate_cluster<3, true>(p, S, per, stream) : launch_gate_cluster<3, false>(p, S, per, stream); break;
            default: e = multi ? launch_gate_cluster<4, true>(p, S, per, stream) : launch_gate_cluster<4, false>(p, S, per, stream); break;
        }
        *launched = 1;
        return e;
    }
    const dim3 pgrid(U, (p.d_gate / 2 + 15) / 16, p.q_len);
    switch (nit) {
        case 1: e = launch_pdl(gate_qproj_kernel<1>, pgrid, dim3(kProjThreads), 0, stream, p); break;
        case 2: e = launch_pdl(gate_qproj_kernel<2>, pgrid, dim3(kProjThreads), 0, stream, p); break;
        case 3: e = launch_pdl(gate_qproj_kernel<3>, pgrid, dim3(kProjThreads), 0, stream, p); break;
        default: e = launch_pdl(gate_qproj_kernel<4>, pgrid, dim3(kProjThreads), 0, stream, p); break;
    }
    if (e != cudaSuccess) return e;
    *launched = 1;
    // slices of about 512 compressed keys, at most 8 per unit
    int S = (p.max_blocks + 511) / 512;
    S = S < 1 ? 1 : (S > 8 ? 8 : S);
    const int per = (p.max_blocks + S - 1) / S;
    e = launch_pdl(gate_score_select_kernel, dim3(S, U), dim3(kGateThreads), 0, stream, p, per);
    if (e != cudaSuccess) return e;
    *launched = 2;
    return cudaGetLastError();
}

}  // namespace seer

// ================================================================================================
// Gate selection without a context: the scratch the split gate kernels need (gate query, block
// scores, per-unit tickets) lives in a fixed array inside the library image instead of a
// context's workspace, for callers that are not allowed to allocate device memory.
// ================================================================================================
#include <mutex>
#include <stdio.h>

#include "../../include/seer.h"

namespace {

// One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[SEER_STATIC_SCRATCH_BYTES];

using seer::kMaxDevices;
std::mutex g_static_mutex;
unsigned char* g_static_ptr[kMaxDevices];     // device address of g_static_scratch, per device

seer_status static_fail(char* err, size_t err_len, seer_status st, const char* fmt, long long a = 0, long long b = 0) {
    if (err && err_len) snprintf(err, err_len, fmt, a, b);
    return st;
}

}  // namespace

extern "C" seer_status seer_gate_select_static(int device, const seer_shape* shape, const seer_gate* gate,
                                               const int32_t* seq_lens, const void* q_nope, int token_budget,
                                               int32_t* block_idx, int32_t* block_cnt, int max_sel,
                                               float* scores_out, void* stream, char* err, size_t err_len) {
    using namespace seer;
    if (err && err_len) err[0] = '\0';
    if (!shape || !gate || !seq_lens || !q_nope || !block_idx || !block_cnt || !gate->w_q || !gate->kcomp)
        return static_fail(err, err_len, SEER_ERR_INVALID_ARG, "NULL pointer among the arguments");
    if (shape->batch <= 0 || shape->num_q_heads <= 0 || shape->num_kv_heads <= 0 || max_sel <= 0 ||
        gate->max_blocks <= 0 || token_budget < 0 || shape->num_q_heads % shape->num_kv_heads != 0)
        return static_fail(err, err_len, SEER_ERR_INVALID_ARG, "sizes must be positive and num_q_heads a multiple of num_kv_heads");
    const int group = shape->num_q_heads / shape->num_kv_heads;
    const int bs = shape->block_size;
    if (shape->head_dim != kHeadDim || (bs != 16 && bs != 32 && bs != 64 && bs != 128) || group > kMaxGroup ||
        (gate->d_gate != 64 && gate->d_gate != 128 && gate->d_gate != 256))
        return static_fail(err, err_len, SEER_ERR_UNSUPPORTED,
                           "supported: head_dim 128, block_size 16/32/64/128, group size <= 8, d_gate 64/128/256");
    if (!(gate->rope_theta > 0.f)) return static_fail(err, err_len, SEER_ERR_INVALID_ARG, "rope_theta must be positive");
    if (((uintptr_t)q_nope | (uintptr_t)gate->w_q | (uintptr_t)gate->kcomp) & 15u)
        return static_fail(err, err_len, SEER_ERR_INVALID_ARG, "q_nope, w_q and kcomp must be 16-byte aligned");
    if (device < 0 || device >= kMaxDevices)
        return static_fail(err, err_len, SEER_ERR_INVALID_ARG, "device index %lld outside 0..%lld", device, kMaxDevices - 1);
    const long long U = (long long)shape->batch * shape->num_kv_heads;
    if (U > 65535) return static_fail(err, err_len, SEER_ERR_UNSUPPORTED, "batch * num_kv_heads above 65535");

    // Layout of the scratch: [status word, 256 B][tickets U ints][gate query U*d_gate floats]
    // [scores U*max_blocks floats].  Only the two-kernel path (more compressed keys per unit than the
    // cluster kernel holds in shared memory) uses anything beyond the status word.
    const bool split = !gate_one_kernel(gate->max_blocks);
    const size_t off_tk = 256;
    const size_t off_qg = off_tk + ((size_t)U * sizeof(int) + 255) / 256 * 256;
    const size_t off_sc = off_qg + ((size_t)U * gate->d_gate * sizeof(float) + 255) / 256 * 256;
    const size_t need = !split ? off_tk : off_sc + (scores_out ? 0 : (size_t)U * gate->max_blocks * sizeof(float));
    if (need > (size_t)SEER_STATIC_SCRATCH_BYTES)
        return static_fail(err, err_len, SEER_ERR_WORKSPACE,
                           "this call needs %lld bytes of scratch, the built-in array holds %lld "
                           "(use seer_gate_select with a context instead)", (long long)need,
                           (long long)SEER_STATIC_SCRATCH_BYTES);

    cudaError_t ce = cudaSetDevice(device);
    if (ce != cudaSuccess) return static_fail(err, err_len, SEER_ERR_CUDA, "cudaSetDevice failed (code %lld)", (long long)ce);
    unsigned char* base = nullptr;
    {
        // once per device, with that device current: the array's name is only a host-side handle,
        // the kernels need its address in this device's memory
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[device]) {
            unsigned char* ptr = nullptr;
            ce = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
            if (ce != cudaSuccess || !ptr)
                return static_fail(err, err_len, SEER_ERR_CUDA, "cudaGetSymbolAddress failed (code %lld)", (long long)ce);
            g_static_ptr[device] = ptr;
        }
        base = g_static_ptr[device];
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the tickets must start at zero (an earlier call may have been cut short); everything else is
    // written before it is read
    if (split) {
        ce = cudaMemsetAsync(base + off_tk, 0, (size_t)U * sizeof(int), s);
        if (ce != cudaSuccess) return static_fail(err, err_len, SEER_ERR_CUDA, "cudaMemsetAsync failed (code %lld)", (long long)ce);
    }

    GateParams p;
    memset(&p, 0, sizeof p);
    p.q_nope = static_cast<const __nv_bfloat16*>(q_nope);
    p.w_q = static_cast<const __nv_bfloat16*>(gate->w_q);
    p.kcomp = static_cast<const __nv_bfloat16*>(gate->kcomp);
    p.seq_lens = seq_lens;
    p.scores_in = nullptr;
    p.scores = scores_out ? scores_out : reinterpret_cast<float*>(base + off_sc);
    p.scores_user = scores_out;
    p.q_gate = reinterpret_cast<float*>(base + off_qg);
    p.block_idx = block_idx;
    p.block_cnt = block_cnt;
    p.batch = shape->batch;
    p.num_q_heads = shape->num_q_heads;
    p.num_kv_heads = shape->num_kv_heads;
    p.group = group;
    p.block_size = shape->block_size;
    p.d_gate = gate->d_gate;
    p.max_blocks = gate->max_blocks;
    p.max_sel = max_sel;
    p.token_budget = token_budget;
    p.q_len = 1;
    p.status = reinterpret_cast<unsigned int*>(base);
    p.tickets = reinterpret_cast<int*>(base + off_tk);
    for (int c = 0; c < gate->d_gate / 2; ++c)
        p.inv_freq[c] = pow((double)gate->rope_theta, -2.0 * (double)c / (double)gate->d_gate);
    int launched = 0;
    ce = launch_gate_select(p, s, &launched);
    if (ce != cudaSuccess) return static_fail(err, err_len, SEER_ERR_CUDA, "kernel launch failed (code %lld)", (long long)ce);
    return SEER_OK;
}
