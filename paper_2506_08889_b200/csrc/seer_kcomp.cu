// K compression cache update (Eq. 1b; Sec. 3.2): per block, max/min/mean pooling of the
// pre-RoPE keys over the block's rows, projection by W_k, RoPE at the block's first token,
// bf16 store.  One CTA handles up to kBlocksPerCta consecutive blocks of one (sequence,
// KV head) so that every W_k element fetched is used for all of them.
#include "seer_device.cuh"
#include "seer_internal.h"

namespace seer {

namespace {

constexpr int kBlocksPerCta = 4;
constexpr int kKcThreads = 256;
constexpr int kMaxDGate = 256;

__global__ void __launch_bounds__(kKcThreads) kcomp_kernel(const KcompParams p) {
    __shared__ float red[kKcThreads / 32][3][kHeadDim];                 // per-warp pooled partials
    __shared__ __align__(16) float feat[kBlocksPerCta][3 * kHeadDim];   // [max | min | avg]
    __shared__ float y[kBlocksPerCta][kMaxDGate];
    __shared__ int blk_of[kBlocksPerCta];

    const int u = blockIdx.y, i = u / p.num_kv_heads, h = u % p.num_kv_heads;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = p.seq_lens[i];
    const int b = p.block_size;
    const int complete = L > 0 ? L / b : 0;           // blocks with all b rows present

    int nb = 0;                                       // blocks this CTA really handles
    int j_first;
    if (p.first_block < 0) {
        j_first = complete - 1;
        nb = (blockIdx.x == 0 && L > 0 && L % b == 0 && j_first < p.max_blocks) ? 1 : 0;
    } else {
        j_first = p.first_block + blockIdx.x * kBlocksPerCta;
        const int j_end = min(min(p.first_block + p.num_blocks, complete), p.max_blocks);
        nb = max(0, min(kBlocksPerCta, j_end - j_first));
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
        for (int r = rgrp; r < b; r += 16) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(
                p.k_nope + base + (row0 + r) * p.stride_token + 8 * cchunk));
            const __nv_bfloat162* hh = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float2 f = __bfloat1622float2(hh[c]);
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
            for (int w2 = 0; w2 < kKcThreads / 32; ++w2) {
                a = fmaxf(a, red[w2][0][tid]);
                m2 = fminf(m2, red[w2][1][tid]);
                s += red[w2][2][tid];
            }
            feat[q][tid] = a;
            feat[q][kHeadDim + tid] = m2;
            feat[q][2 * kHeadDim + tid] = s / (float)b;
        }
        if (tid == 0) blk_of[q] = j;
        __syncthreads();
    }
    for (int q = nb; q < kBlocksPerCta; ++q)
        for (int c = tid; c < 3 * kHeadDim; c += kKcThreads) feat[q][c] = 0.f;
    __syncthreads();

    // projection: one warp per output row, all blocks of the CTA at once
    const int in_chunks = 3 * kHeadDim / 8;           // 48 x 16 B per W_k row
    for (int r = warp; r < p.d_gate; r += kKcThreads / 32) {
        const uint4* wrow = reinterpret_cast<const uint4*>(p.w_k + ((size_t)h * p.d_gate + r) * 3 * kHeadDim);
        float acc[kBlocksPerCta];
#pragma unroll
        for (int q = 0; q < kBlocksPerCta; ++q) acc[q] = 0.f;
        for (int ch = lane; ch < in_chunks; ch += 32) {
            const uint4 wv = __ldg(wrow + ch);
            const __nv_bfloat162* hh = reinterpret_cast<const __nv_bfloat162*>(&wv);
            float wf[8];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float2 f = __bfloat1622float2(hh[c]);
                wf[2 * c] = f.x; wf[2 * c + 1] = f.y;
            }
#pragma unroll
            for (int q = 0; q < kBlocksPerCta; ++q) {
                const float4 f0 = *reinterpret_cast<const float4*>(&feat[q][8 * ch]);
                const float4 f1 = *reinterpret_cast<const float4*>(&feat[q][8 * ch + 4]);
                acc[q] = fmaf(wf[0], f0.x, acc[q]); acc[q] = fmaf(wf[1], f0.y, acc[q]);
                acc[q] = fmaf(wf[2], f0.z, acc[q]); acc[q] = fmaf(wf[3], f0.w, acc[q]);
                acc[q] = fmaf(wf[4], f1.x, acc[q]); acc[q] = fmaf(wf[5], f1.y, acc[q]);
                acc[q] = fmaf(wf[6], f1.z, acc[q]); acc[q] = fmaf(wf[7], f1.w, acc[q]);
            }
        }
#pragma unroll
        for (int q = 0; q < kBlocksPerCta; ++q) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], off);
        }
        if (lane == 0) {
#pragma unroll
            for (int q = 0; q < kBlocksPerCta; ++q) y[q][r] = acc[q];
        }
    }
    __syncthreads();

    // RoPE at the position of the block's first token, then the bf16 store
    const int half = p.d_gate / 2;
    for (int x = tid; x < nb * half; x += kKcThreads) {
        const int q = x / half, c = x % half;
        const int j = blk_of[q];
        const double ang = (double)j * (double)b * pow((double)p.rope_theta, -2.0 * (double)c / (double)p.d_gate);
        double sn, cs;
        sincos(ang, &sn, &cs);
        const double a = y[q][c], bb = y[q][c + half];
        __nv_bfloat16* dst = p.kcomp + ((size_t)u * p.max_blocks + j) * p.d_gate;
        dst[c] = __double2bfloat16(a * cs - bb * sn);
        dst[c + half] = __double2bfloat16(bb * cs + a * sn);
    }
}

}  // namespace

cudaError_t launch_kcomp_append(const KcompParams& p, cudaStream_t stream, int* launched) {
    const int U = p.batch * p.num_kv_heads;
    const int gx = p.first_block < 0 ? 1 : (p.num_blocks + kBlocksPerCta - 1) / kBlocksPerCta;
    *launched = 0;
    if (gx <= 0 || U <= 0) return cudaSuccess;
    kcomp_kernel<<<dim3(gx, U), kKcThreads, 0, stream>>>(p);
    *launched = 1;
    return cudaGetLastError();
}

}  // namespace seer
