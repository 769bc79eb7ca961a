// AttnGate at decode time (Eq. 1a, 1c; Sec. 3.1): Q-branch projection + RoPE, block scores
// against the K compression cache, and the token-budget top-k with the forced last block.
#include "seer_device.cuh"
#include "seer_internal.h"

namespace seer {

namespace {

__device__ __forceinline__ float dot8(const uint4& a, const float* x) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&a);
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        float2 f = __bfloat1622float2(h[k]);
        acc = fmaf(f.x, x[2 * k], acc);
        acc = fmaf(f.y, x[2 * k + 1], acc);
    }
    return acc;
}

// ---- q_gate = RoPE_{L_i - 1}( W_q[h] . concat_g(Q_nope) ) ----------------------------------
// grid (B*Hkv, ceil(dg/2 / 4)), 128 threads; each warp computes one rotary pair (c, c + dg/2).
__global__ void __launch_bounds__(128) gate_qproj_kernel(const GateParams p) {
    __shared__ float x[kMaxGroup * kHeadDim];
    const int u = blockIdx.x, i = u / p.num_kv_heads, h = u % p.num_kv_heads;
    const int n = p.group * kHeadDim;
    const __nv_bfloat16* src = p.q_nope + ((size_t)i * p.num_q_heads + (size_t)h * p.group) * kHeadDim;
    for (int c = threadIdx.x; c < n; c += blockDim.x) x[c] = __bfloat162float(src[c]);
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int half = p.d_gate / 2;
    const int c = blockIdx.y * 4 + warp;
    if (c >= half) return;
    const __nv_bfloat16* w0 = p.w_q + ((size_t)h * p.d_gate + c) * n;
    const __nv_bfloat16* w1 = p.w_q + ((size_t)h * p.d_gate + c + half) * n;
    float a0 = 0.f, a1 = 0.f;
    for (int ch = lane; ch < n / 8; ch += 32) {
        const uint4 v0 = __ldg(reinterpret_cast<const uint4*>(w0) + ch);
        const uint4 v1 = __ldg(reinterpret_cast<const uint4*>(w1) + ch);
        a0 += dot8(v0, x + 8 * ch);
        a1 += dot8(v1, x + 8 * ch);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        a0 += __shfl_xor_sync(0xffffffffu, a0, off);
        a1 += __shfl_xor_sync(0xffffffffu, a1, off);
    }
    if (lane == 0) {
        const int L = p.seq_lens[i];
        const double pos = (double)(L > 0 ? L - 1 : 0);
        const double ang = pos * pow((double)p.rope_theta, -2.0 * (double)c / (double)p.d_gate);
        double sn, cs;
        sincos(ang, &sn, &cs);
        float* dst = p.q_gate + (size_t)u * p.d_gate;
        dst[c] = (float)((double)a0 * cs - (double)a1 * sn);
        dst[c + half] = (float)((double)a1 * cs + (double)a0 * sn);
    }
}

// ---- score[j] = <q_gate, Kc[j]> / sqrt(dg) for j < n_i - 1 ----------------------------------
// grid (ceil(max_blocks / 64), B*Hkv), 128 threads; 16 lanes per block entry.
__global__ void __launch_bounds__(128) gate_scores_kernel(const GateParams p) {
    __shared__ float qg[256];
    const int u = blockIdx.y, i = u / p.num_kv_heads;
    const int L = p.seq_lens[i];
    const int n_i = (L + p.block_size - 1) / p.block_size;
    const int n_cand = min(n_i - 1, p.max_blocks);
    const int j0 = blockIdx.x * 64;
    if (j0 >= n_cand) return;
    for (int c = threadIdx.x; c < p.d_gate; c += blockDim.x) qg[c] = p.q_gate[(size_t)u * p.d_gate + c];
    __syncthreads();
    const int sub = threadIdx.x & 15, grp = threadIdx.x >> 4;       // 8 groups of 16 lanes
    const float inv = rsqrtf((float)p.d_gate);
    const int chunks = p.d_gate / 8;
    for (int jj = grp; jj < 64; jj += 8) {
        const int j = j0 + jj;
        const bool live = j < n_cand;
        float acc = 0.f;
        if (live) {
            const uint4* row = reinterpret_cast<const uint4*>(p.kcomp + ((size_t)u * p.max_blocks + j) * p.d_gate);
            for (int ch = sub; ch < chunks; ch += 16) acc += dot8(__ldg(row + ch), qg + 8 * ch);
        }
#pragma unroll
        for (int off = 8; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (live && sub == 0) p.scores[(size_t)u * p.max_blocks + j] = acc * inv;
    }
}

// ---- token-budget selection ------------------------------------------------------------------
// Order-preserving key: larger score <-> larger key; -0 == +0; NaN below everything.
__device__ __forceinline__ uint32_t score_key(float s) {
    if (s != s) return 0u;
    uint32_t b = __float_as_uint(s);
    if (b == 0x80000000u) b = 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

constexpr int kSelThreads = 256;

// One CTA per (sequence, KV head).  Radix select (4 passes of 8 bits) finds the key of the
// (k-1)-th best candidate; a final ordered pass emits, in ascending block order, every
// candidate above it plus the first few equal to it (lower block number wins a tie), then
// the forced last block.  Comparisons only: the result is exact.
__global__ void __launch_bounds__(kSelThreads) gate_topk_kernel(const GateParams p) {
    __shared__ int hist[256];
    __shared__ int warp_cnt[2][kSelThreads / 32];
    __shared__ uint32_t sh_prefix;
    __shared__ int sh_need;
    const int u = blockIdx.x, i = u / p.num_kv_heads;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t* dst = p.block_idx + (size_t)u * p.max_sel;
    const float* sc = (p.scores_in ? p.scores_in : p.scores) + (size_t)u * p.max_blocks;
    const int L = p.seq_lens[i];
    const int n_i = L > 0 ? (L + p.block_size - 1) / p.block_size : 0;
    if (n_i <= 0) {
        for (int e = tid; e < p.max_sel; e += kSelThreads) dst[e] = -1;
        if (tid == 0) p.block_cnt[u] = 0;
        return;
    }
    int k = p.token_budget / p.block_size;
    k = max(k, 1);
    k = min(k, min(n_i, p.max_sel));
    const int n_cand = min(n_i - 1, p.max_blocks);
    int need = min(k - 1, n_cand);          // candidates to take besides the last block

    uint32_t thr = 0u;                      // key of the need-th best candidate
    int take_eq = 0;                        // how many candidates equal to thr to take
    if (need > 0 && need < n_cand) {
        uint32_t prefix = 0u;
        int rem = need;
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            const uint32_t himask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
            for (int b = tid; b < 256; b += kSelThreads) hist[b] = 0;
            __syncthreads();
            for (int j = tid; j < n_cand; j += kSelThreads) {
                const uint32_t key = score_key(sc[j]);
                if ((key & himask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
            }
            __syncthreads();
            if (tid == 0) {
                int acc = 0, b = 255;
                for (; b > 0; --b) {
                    if (acc + hist[b] >= rem) break;
                    acc += hist[b];
                }
                sh_prefix = prefix | ((uint32_t)b << shift);
                sh_need = rem - acc;
            }
            __syncthreads();
            prefix = sh_prefix;
            rem = sh_need;
        }
        thr = prefix;
        take_eq = rem;
    } else if (need >= n_cand) {
        thr = 0u;                           // everything qualifies: key >= 0 always
        take_eq = n_cand;
        need = n_cand;
    }

    // ordered emission
    int out_base = 0, eq_base = 0;
    if (need > 0) {
        for (int j0 = 0; j0 < n_cand; j0 += kSelThreads) {
            const int j = j0 + tid;
            uint32_t key = 0u;
            const bool live = j < n_cand;
            if (live) key = score_key(sc[j]);
            const bool gt = live && key > thr;
            const bool eq = live && key == thr;
            const unsigned bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
            if (lane == 0) { warp_cnt[0][warp] = __popc(bg); warp_cnt[1][warp] = __popc(be); }
            __syncthreads();
            int gt_before = 0, eq_before = 0, gt_total = 0, eq_total = 0;
#pragma unroll
            for (int w2 = 0; w2 < kSelThreads / 32; ++w2) {
                const int a = warp_cnt[0][w2], b = warp_cnt[1][w2];
                if (w2 < warp) { gt_before += a; eq_before += b; }
                gt_total += a; eq_total += b;
            }
            const unsigned lt_mask = (1u << lane) - 1u;
            gt_before += __popc(bg & lt_mask);
            eq_before += __popc(be & lt_mask);
            // equal-key candidates are taken in index order until take_eq are in
            const int eq_rank = eq_base + eq_before;
            const int eq_taken_before = min(eq_rank, take_eq);
            const bool sel = gt || (eq && eq_rank < take_eq);
            if (sel) dst[out_base + gt_before + eq_taken_before - min(eq_base, take_eq)] = j;
            out_base += gt_total + (min(eq_base + eq_total, take_eq) - min(eq_base, take_eq));
            eq_base += eq_total;
            __syncthreads();
        }
    }
    // forced last block, padding, count
    if (tid == 0) {
        dst[need] = n_i - 1;
        p.block_cnt[u] = need + 1;
    }
    for (int e = need + 1 + tid; e < p.max_sel; e += kSelThreads) dst[e] = -1;
}

}  // namespace

cudaError_t launch_gate_select(const GateParams& p, cudaStream_t stream, int* launched) {
    const int U = p.batch * p.num_kv_heads;
    *launched = 0;
    if (!p.scores_in) {
        const int half = p.d_gate / 2;
        gate_qproj_kernel<<<dim3(U, (half + 3) / 4), 128, 0, stream>>>(p);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        gate_scores_kernel<<<dim3((p.max_blocks + 63) / 64, U), 128, 0, stream>>>(p);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        *launched += 2;
    }
    gate_topk_kernel<<<U, kSelThreads, 0, stream>>>(p);
    *launched += 1;
    return cudaGetLastError();
}

}  // namespace seer
