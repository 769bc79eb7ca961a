// C ABI of the library: context, argument validation, tensor-map construction, launches.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "../../include/seer.h"
#include "seer_device.cuh"
#include "seer_internal.h"

using namespace seer;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

struct MapKey {
    const void* base;
    uint64_t dims[4];
    uint64_t strides[3];
    uint64_t box_rows;
    bool operator==(const MapKey& o) const { return memcmp(this, &o, sizeof(MapKey)) == 0; }
};

constexpr int kMapCache = 256;            // tensor-map cache slots (K and V of 128 layers), open addressing
constexpr int kMapProbe = 8;              // slots looked at per lookup

}  // namespace

struct seer_ctx {
    int device;
    int num_sms;
    unsigned char* ws;          // device workspace
    size_t ws_bytes;
    EncodeTiledFn encode;
    MapKey map_keys[kMapCache];
    CUtensorMap maps[kMapCache];
    bool map_valid[kMapCache];
    uint64_t launches;
    unsigned int generation;    // stamps the partials of a decode launch
    int pool_div;               // decode scheduling: share of tiles handed out dynamically
    int min_tiles;              // decode scheduling: fewest tiles of a CTA's range
    int sel_from_lens;          // set by seer_decode_step around its attention call (see DecodeParams)
    int list_gen;               // != 0 inside seer_decode_step: the gate marks finished lists with it, the attention kernel waits per unit
    int list_gen_last;          // the last such number handed out
    int use_list_flags;         // 0: the attention kernel of a step waits for the whole gate kernel instead (SEER_STEP_LIST_FLAGS=0)
    int wide_variant;           // kernel variant code for more than 16 rows per unit: 16 (tcgen05), 8 (mma.sync), 0 (by size)
    char err[512];
};

namespace {

constexpr size_t kStatusBytes = 256;

seer_status fail(seer_ctx* ctx, seer_status s, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof ctx->err, fmt, ap);
        va_end(ap);
    }
    return s;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Workspace: [status][scheduler counters][decode tickets][gate tickets] at fixed offsets, then one
// scratch region that a decode call uses for its partials and a gate call for its gate query and
// scores (calls on a context are ordered, and neither kind of scratch outlives its call).
constexpr int kMaxGridCtas = 148 * 2 * 4;   // generous bound on the decode grid, for workspace sizing

struct WsLayout {
    size_t sched, steal, tickets, gate_tickets, list_flags, prefix, scratch;
    size_t part_o, part_ml, q_gate, scores, total;
};

constexpr int kMaxUnits = 65535;            // batch * num_kv_heads (check_shape enforces it)

WsLayout ws_layout(int num_units, int slots, int d_gate, int max_blocks, int n_tiles = 1) {
    WsLayout w;
    // The regions that must stay zero between launches sit at offsets that do not depend on the
    // call's shape (they are sized for the largest unit count), so that calls of different shapes on
    // one context never see one another's scratch in them.
    size_t off = kStatusBytes;
    w.sched = off; off += 256;
    w.steal = off; off = align_up(off + sizeof(int) * (size_t)kMaxGridCtas, 256);
    w.tickets = off; off = align_up(off + sizeof(unsigned long long) * (size_t)kMaxUnits, 256);
    w.gate_tickets = off; off = align_up(off + sizeof(int) * (size_t)kMaxUnits, 256);
    w.list_flags = off; off = align_up(off + sizeof(int) * (size_t)kMaxUnits, 256);
    w.prefix = off; off = align_up(off + sizeof(int) * ((size_t)kMaxUnits + 1), 256);
    w.scratch = off;
    // decode view of the scratch
    size_t d = off;
    w.part_ml = d; d = align_up(d + sizeof(float) * (size_t)slots * 32 * n_tiles, 256);
    w.part_o = d;  d = align_up(d + sizeof(float) * (size_t)slots * 8 * n_tiles * kHeadDim, 256);
    // gate view of the scratch
    size_t g = off;
    w.q_gate = g;  g = align_up(g + sizeof(float) * (size_t)num_units * 8 /* query tokens */ * (size_t)(d_gate > 0 ? d_gate : 0), 256);
    w.scores = g;  g = align_up(g + sizeof(float) * (size_t)num_units * (size_t)(max_blocks > 0 ? max_blocks : 0), 256);
    w.total = d > g ? d : g;
    return w;
}


seer_status check_shape(seer_ctx* ctx, const seer_shape* s) {
    if (!s) return fail(ctx, SEER_ERR_INVALID_ARG, "shape is NULL");
    if (s->batch <= 0 || s->num_q_heads <= 0 || s->num_kv_heads <= 0)
        return fail(ctx, SEER_ERR_INVALID_ARG, "batch/head counts must be positive");
    if (s->head_dim != kHeadDim) return fail(ctx, SEER_ERR_UNSUPPORTED, "head_dim %d (only 128)", s->head_dim);
    if (s->block_size != 16 && s->block_size != 32 && s->block_size != 64 && s->block_size != 128)
        return fail(ctx, SEER_ERR_UNSUPPORTED, "block_size %d (only 16, 32, 64 or 128)", s->block_size);
    if (s->num_q_heads % s->num_kv_heads != 0)
        return fail(ctx, SEER_ERR_INVALID_ARG, "num_q_heads %d not a multiple of num_kv_heads %d",
                    s->num_q_heads, s->num_kv_heads);
    const int g = s->num_q_heads / s->num_kv_heads;
    if (g < 1 || g > kMaxGroup) return fail(ctx, SEER_ERR_UNSUPPORTED, "group size %d (supported 1..8)", g);
    if ((long long)s->batch * s->num_kv_heads > 65535)
        return fail(ctx, SEER_ERR_UNSUPPORTED, "batch * num_kv_heads above 65535");
    return SEER_OK;
}

// Rotary frequencies theta^(-2c/d_gate) in double (the device only multiplies by the position).
void fill_inv_freq(double* dst, int d_gate, float theta) {
    for (int c = 0; c < d_gate / 2; ++c) dst[c] = pow((double)theta, -2.0 * (double)c / (double)d_gate);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

seer_status get_map(seer_ctx* ctx, const void* base, const uint64_t dims[4], const uint64_t strides_bytes[3],
                    int box_rows, const CUtensorMap** out) {
    MapKey key;
    memset(&key, 0, sizeof key);
    key.base = base;
    for (int a = 0; a < 4; ++a) key.dims[a] = dims[a];
    for (int a = 0; a < 3; ++a) key.strides[a] = strides_bytes[a];
    key.box_rows = (uint64_t)box_rows;
    // hashed on the base address (a layer's K or V cache), a few slots probed; a full neighbourhood
    // gives up its first slot
    const uint64_t hb = reinterpret_cast<uintptr_t>(base) >> 8;
    const int home = (int)((hb ^ (hb >> 11) ^ (hb >> 23)) & (kMapCache - 1));
    int slot = -1;
    for (int a = 0; a < kMapProbe; ++a) {
        const int c = (home + a) & (kMapCache - 1);
        if (ctx->map_valid[c]) {
            if (ctx->map_keys[c] == key) { *out = &ctx->maps[c]; return SEER_OK; }
        } else if (slot < 0) {
            slot = c;
        }
    }
    if (slot < 0) slot = home;
    ctx->map_valid[slot] = false;
    cuuint64_t gd[4] = {dims[0], dims[1], dims[2], dims[3]};
    cuuint64_t gs[3] = {strides_bytes[0], strides_bytes[1], strides_bytes[2]};
    cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};          // 64 channels (128 B) x 64 tokens (or one small block)
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = ctx->encode(&ctx->maps[slot], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), gd, gs,
                             box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ctx, SEER_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    ctx->map_keys[slot] = key;
    ctx->map_valid[slot] = true;
    *out = &ctx->maps[slot];
    return SEER_OK;
}

seer_status decode_common(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv, const void* q, int q_len,
                          const int32_t* block_idx, const int32_t* block_cnt, int max_sel, bool sparse,
                          void* out, float* lse, void* stream) {
    if (!ctx) return SEER_ERR_INVALID_ARG;
    seer_status st = check_shape(ctx, shape);
    if (st != SEER_OK) return st;
    if (!kv || !kv->k || !kv->v || !kv->seq_lens || !q || !out)
        return fail(ctx, SEER_ERR_INVALID_ARG, "NULL pointer among kv/k/v/seq_lens/q/out");
    if (!aligned16(kv->k) || !aligned16(kv->v) || !aligned16(q) || !aligned16(out))
        return fail(ctx, SEER_ERR_INVALID_ARG, "k, v, q and out must be 16-byte aligned");
    if (kv->stride_batch % 8 || kv->stride_head % 8 || kv->stride_token % 8 || kv->stride_batch <= 0 ||
        kv->stride_head <= 0 || kv->stride_token < kHeadDim)
        return fail(ctx, SEER_ERR_INVALID_ARG, "K/V strides must be positive multiples of 8 elements");
    if (kv->max_seq_len <= 0) return fail(ctx, SEER_ERR_INVALID_ARG, "max_seq_len must be positive");
    if (q_len < 1 || q_len > 8) return fail(ctx, SEER_ERR_UNSUPPORTED, "q_len %d (supported 1..8)", q_len);
    const bool paged = kv->page_table != nullptr;
    if (paged) {
        if (kv->page_size <= 0 || kv->page_size % kTileTokens != 0)
            return fail(ctx, SEER_ERR_UNSUPPORTED, "page_size %d (must be a multiple of 64)", kv->page_size);
        if (kv->num_pages <= 0 || kv->page_table_stride <= 0)
            return fail(ctx, SEER_ERR_INVALID_ARG, "num_pages and page_table_stride must be positive");
        if ((long long)kv->page_table_stride * kv->page_size < kv->max_seq_len)
            return fail(ctx, SEER_ERR_INVALID_ARG, "page table row shorter than max_seq_len");
    }
    if (sparse) {
        if (!block_idx) return fail(ctx, SEER_ERR_INVALID_ARG, "block_idx is NULL");
        if (max_sel <= 0) return fail(ctx, SEER_ERR_INVALID_ARG, "max_sel must be positive");
    }
    const int U = shape->batch * shape->num_kv_heads;
    // blocks of 64 or 128 tokens are one or two tiles; blocks of 16 or 32 tokens are gathered 4 or 2 to a tile
    const int bpt = shape->block_size < kTileTokens ? kTileTokens / shape->block_size : 1;
    const int tpb = bpt > 1 ? 1 : shape->block_size / kTileTokens;

    cudaError_t ce = cudaSetDevice(ctx->device);
    if (ce != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "cudaSetDevice: %s", cudaGetErrorString(ce));
    // A decode launch carries counters that the host advances per call (the stamp of its partial results, the
    // number its step's list marks must show): replayed from a captured graph they would repeat, and partials or
    // marks left by the previous replay would pass for this one's.  Refuse rather than compute wrong results.
    {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(static_cast<cudaStream_t>(stream), &cap) == cudaSuccess && cap != cudaStreamCaptureStatusNone)
            return fail(ctx, SEER_ERR_UNSUPPORTED,
                        "the stream is being captured: decode launches carry per-call counters and cannot be replayed from a graph");
    }
    // Query tokens share a launch while (tokens x group) fits the kernel's 16 rows; more tokens
    // take further launches over the same lists (each reads the selected K/V once).
    // Up to 16 rows ride on the MMA's N side (tokens on M); more than 16 rows (with blocks of 64 or 128 tokens)
    // take the variant with the rows on M, up to 64 a launch.
    const int group = shape->num_q_heads / shape->num_kv_heads;
    const bool wide = q_len * group > 16 && bpt == 1;
    const int row_cap = wide ? 64 : 16;
    const int tok_per_launch = q_len < row_cap / group ? q_len : row_cap / group;
    const int n_tiles = wide ? 8 : tok_per_launch * group > 8 ? 2 : 1;    // (sizes the partial slots: 8 rows each)
    // (the kernel: 16 = rows on M by tcgen05, the faster one up to 48 rows; 8 = rows on M by mma.sync)
    const int variant = !wide ? n_tiles : ctx->wide_variant ? ctx->wide_variant : tok_per_launch * group <= 48 ? 16 : 8;
    const int per_sm = decode_ctas_per_sm(sparse, paged, variant);
    if (per_sm <= 0) return fail(ctx, SEER_ERR_CUDA, "decode kernel cannot be resident (shared memory)");
    long long max_tiles = sparse ? (long long)U * ((max_sel + bpt - 1) / bpt) * tpb
                                 : (long long)U * ((kv->max_seq_len + kTileTokens - 1) / kTileTokens);
    int grid = ctx->num_sms * per_sm;
    if (grid > kMaxGridCtas) grid = kMaxGridCtas;
    if (max_tiles < grid) grid = (int)(max_tiles > 0 ? max_tiles : 1);
    // a partial slot of the wide variant is 33 KiB: fewer dynamic chunks per range if the workspace asks for it
    int max_rounds = kMaxRounds;
    WsLayout w = ws_layout(U, decode_max_intervals(grid, max_rounds) + U, 0, 0, n_tiles);
    while (w.total > ctx->ws_bytes && max_rounds > 0) {
        --max_rounds;
        w = ws_layout(U, decode_max_intervals(grid, max_rounds) + U, 0, 0, n_tiles);
    }
    if (w.total > ctx->ws_bytes)
        return fail(ctx, SEER_ERR_WORKSPACE, "workspace %zu bytes, call needs %zu", ctx->ws_bytes, w.total);

    // tensor maps: (channel, token row, head, sequence-or-page)
    const uint64_t rows = paged ? (uint64_t)kv->page_size : (uint64_t)kv->max_seq_len;
    const uint64_t outer = paged ? (uint64_t)kv->num_pages : (uint64_t)shape->batch;
    const uint64_t dims[4] = {(uint64_t)kHeadDim, rows, (uint64_t)shape->num_kv_heads, outer};
    const uint64_t strides[3] = {(uint64_t)kv->stride_token * 2, (uint64_t)kv->stride_head * 2,
                                 (uint64_t)kv->stride_batch * 2};
    const CUtensorMap *mk, *mv;
    const int box_rows = sparse && bpt > 1 ? shape->block_size : kTileTokens;
    st = get_map(ctx, kv->k, dims, strides, box_rows, &mk);
    if (st != SEER_OK) return st;
    const CUtensorMap mk_copy = *mk;       // the second lookup may evict the first
    st = get_map(ctx, kv->v, dims, strides, box_rows, &mv);
    if (st != SEER_OK) return st;

    DecodeParams p;
    memset(&p, 0, sizeof p);
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    p.seq_lens = kv->seq_lens;
    p.block_idx = block_idx;
    p.block_cnt = block_cnt;
    p.page_table = kv->page_table;
    p.page_table_stride = kv->page_table_stride;
    p.max_sel = max_sel;
    p.sel_from_lens = sparse && q_len == 1 ? ctx->sel_from_lens : 0;
    if (p.sel_from_lens > 0 && ctx->list_gen != 0) {
        p.list_flags = reinterpret_cast<const int*>(ctx->ws + w.list_flags);
        p.list_gen = ctx->list_gen;
    }
    p.page_size = kv->page_size;
    p.num_pages = kv->num_pages;
    p.batch = shape->batch;
    p.num_q_heads = shape->num_q_heads;
    p.num_kv_heads = shape->num_kv_heads;
    p.group = group;
    p.q_len = q_len;
    p.block_size = shape->block_size;
    p.tiles_per_block = tpb;
    p.blocks_per_tile = bpt;
    p.bs_shift = shape->block_size == 16 ? 4 : shape->block_size == 32 ? 5 : shape->block_size == 64 ? 6 : 7;
    p.tpb_shift = tpb == 2 ? 1 : 0;
    p.bpt_shift = bpt == 4 ? 2 : bpt == 2 ? 1 : 0;
    p.kvh_magic = shape->num_kv_heads == 1 ? 0u
                                           : (unsigned int)((0x100000000ull + (unsigned long long)shape->num_kv_heads - 1) /
                                                            (unsigned long long)shape->num_kv_heads);
    p.group_magic = (65536 + group - 1) / group;
    p.num_units = U;
    p.max_blocks_cap = (kv->max_seq_len + kTileTokens - 1) / kTileTokens;
    p.pool_div = ctx->pool_div;
    p.min_tiles = ctx->min_tiles;
    p.max_rounds = max_rounds;
    p.scale_log2 = shape->sm_scale * 1.4426950408889634f;
    p.status = reinterpret_cast<unsigned int*>(ctx->ws);
    p.tickets = reinterpret_cast<unsigned long long*>(ctx->ws + w.tickets);
    p.sched = reinterpret_cast<int*>(ctx->ws + w.sched);
    p.prefix = reinterpret_cast<int*>(ctx->ws + w.prefix);
    p.steal = reinterpret_cast<int*>(ctx->ws + w.steal);
    p.part_o = reinterpret_cast<float*>(ctx->ws + w.part_o);
    p.part_ml = reinterpret_cast<float*>(ctx->ws + w.part_ml);

#ifdef SEER_DECODE_TRACE
    p.trace = reinterpret_cast<unsigned long long*>(ctx->ws + (ctx->ws_bytes - (size_t)(1 << 20)));
#endif
    for (int t0 = 0; t0 < q_len; t0 += tok_per_launch) {
        p.t_base = t0;
        p.t_cnt = q_len - t0 < tok_per_launch ? q_len - t0 : tok_per_launch;
        p.rows = p.t_cnt * group;
        p.generation = ++ctx->generation;
        ce = launch_decode(sparse, paged, variant, mk_copy, *mv, p, grid, static_cast<cudaStream_t>(stream));
        if (ce != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "decode launch: %s", cudaGetErrorString(ce));
        ctx->launches += 1;
    }
    return SEER_OK;
}

}  // namespace

extern "C" {

seer_status seer_create(seer_ctx** out, int device, size_t workspace_bytes) {
    if (!out) return SEER_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return SEER_ERR_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return SEER_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SEER_ERR_CUDA;
    if (prop.major != 10) return SEER_ERR_UNSUPPORTED;    // kernels are built for sm_100a only
    seer_ctx* ctx = new (std::nothrow) seer_ctx;
    if (!ctx) return SEER_ERR_CUDA;
    memset(ctx, 0, sizeof *ctx);
    ctx->device = device;
    ctx->num_sms = prop.multiProcessorCount;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) {
        delete ctx;
        return SEER_ERR_CUDA;
    }
    ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
    ctx->pool_div = 4;
    if (const char* e = getenv("SEER_DECODE_POOL_DIV")) ctx->pool_div = atoi(e);
    ctx->min_tiles = 4;
    if (const char* e = getenv("SEER_DECODE_MIN_TILES")) ctx->min_tiles = atoi(e);
    ctx->use_list_flags = 1;
    if (const char* e = getenv("SEER_STEP_LIST_FLAGS")) ctx->use_list_flags = atoi(e) != 0;
    ctx->wide_variant = 0;      // chosen by the number of rows
    if (const char* e = getenv("SEER_DECODE_WIDE_VARIANT")) ctx->wide_variant = atoi(e) == 16 ? 16 : atoi(e) == 8 ? 8 : 0;
    ctx->ws_bytes = workspace_bytes ? workspace_bytes : (size_t)64 << 20;
    if (ctx->ws_bytes < 4096) ctx->ws_bytes = 4096;     // (far too small for any call: every call checks)
    if (cudaMalloc(reinterpret_cast<void**>(&ctx->ws), ctx->ws_bytes) != cudaSuccess) {
        delete ctx;
        return SEER_ERR_CUDA;
    }
    if (cudaMemset(ctx->ws, 0, ctx->ws_bytes) != cudaSuccess) {
        cudaFree(ctx->ws);
        delete ctx;
        return SEER_ERR_CUDA;
    }
    *out = ctx;
    return SEER_OK;
}

void seer_destroy(seer_ctx* ctx) {
    if (!ctx) return;
    cudaSetDevice(ctx->device);
    cudaFree(ctx->ws);
    delete ctx;
}

const char* seer_status_string(seer_status s) {
    switch (s) {
        case SEER_OK: return "ok";
        case SEER_ERR_INVALID_ARG: return "invalid argument";
        case SEER_ERR_UNSUPPORTED: return "unsupported shape";
        case SEER_ERR_WORKSPACE: return "workspace too small";
        case SEER_ERR_CUDA: return "CUDA error";
        case SEER_ERR_BAD_INDEX: return "block index or page id out of range (skipped)";
        case SEER_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

const char* seer_last_error(const seer_ctx* ctx) { return ctx ? ctx->err : "context is NULL"; }

uint64_t seer_launch_count(const seer_ctx* ctx) { return ctx ? ctx->launches : 0; }

#ifdef SEER_DECODE_TRACE
/* diagnostic builds only: device address of the per-CTA time stamps of the last decode launch */
void* seer_debug_trace_ptr(seer_ctx* ctx) { return ctx->ws + (ctx->ws_bytes - (size_t)(1 << 20)); }
int seer_debug_ctas_per_sm(int sparse, int paged) { return decode_ctas_per_sm(sparse != 0, paged != 0, 1); }
#endif

namespace {
// One CTA waits, with the given poll limit, on an mbarrier that nobody ever arrives at, gives up, raises
// DEV_TIMEOUT as the library's kernels do, and leaves the counters that a kernel cut short would leave
// (a ticket, the scheduler words, a claim counter) non-zero.
__global__ void debug_wait_timeout_kernel(unsigned int* status, unsigned long long* tickets, int* sched, int* steal,
                                          unsigned int polls) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
    }
    __syncthreads();
    if (threadIdx.x == 0 && !mbar_wait(&bar, 0, status, polls)) {
        tickets[0] = (3ull << 32) | 5ull;
        sched[0] = 7;
        sched[1] = 2;
        steal[1] = 1 | (1 << 16);
    }
}

// Reads n16 16-byte words once, eight loads in flight per thread, and folds their 32-bit words into one
// checksum (so that no load can be dropped): what a kernel that only reads can get out of the memory.
constexpr int kProbeThreads = 512;
__global__ void __launch_bounds__(kProbeThreads, 2) read_probe_kernel(const uint4* __restrict__ src, size_t n16,
                                                                    unsigned long long* checksum) {
    const size_t stride = (size_t)gridDim.x * kProbeThreads;
    size_t i = (size_t)blockIdx.x * kProbeThreads + threadIdx.x;
    uint4 acc = make_uint4(0u, 0u, 0u, 0u);
    for (; i + 7 * stride < n16; i += 8 * stride) {
        uint4 v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = __ldcs(src + i + k * stride);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            acc.x ^= v[k].x;
            acc.y ^= v[k].y;
            acc.z ^= v[k].z;
            acc.w ^= v[k].w;
        }
    }
    for (; i < n16; i += stride) {
        const uint4 v = __ldcs(src + i);
        acc.x ^= v.x;
        acc.y ^= v.y;
        acc.z ^= v.z;
        acc.w ^= v.w;
    }
    unsigned int x = acc.x ^ acc.y ^ acc.z ^ acc.w;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x ^= __shfl_xor_sync(0xffffffffu, x, o);
    if ((threadIdx.x & 31) == 0 && x != 0u) atomicXor(checksum, (unsigned long long)x);
}
}  // namespace

seer_status seer_debug_read_bandwidth(seer_ctx* ctx, const void* src, size_t bytes, unsigned long long* checksum,
                                      void* stream) {
    if (!ctx) return SEER_ERR_INVALID_ARG;
    if (!src || !checksum) return fail(ctx, SEER_ERR_INVALID_ARG, "src or checksum is NULL");
    if ((reinterpret_cast<uintptr_t>(src) & 15) || (bytes & 15) || (reinterpret_cast<uintptr_t>(checksum) & 7))
        return fail(ctx, SEER_ERR_INVALID_ARG, "src and bytes must be multiples of 16, checksum 8-byte aligned");
    cudaError_t ce = cudaSetDevice(ctx->device);
    if (ce != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "cudaSetDevice: %s", cudaGetErrorString(ce));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    ce = cudaMemsetAsync(checksum, 0, sizeof(unsigned long long), s);
    if (ce != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "memset: %s", cudaGetErrorString(ce));
    if (bytes == 0) return SEER_OK;
    const size_t n16 = bytes / 16;
    size_t grid = (n16 + kProbeThreads - 1) / kProbeThreads;
    const size_t full = (size_t)ctx->num_sms * 2;
    if (grid > full) grid = full;
    read_probe_kernel<<<(unsigned int)grid, kProbeThreads, 0, s>>>(static_cast<const uint4*>(src), n16, checksum);
    ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "launch: %s", cudaGetErrorString(ce));
    ctx->launches += 1;
    return SEER_OK;
}

seer_status seer_debug_wait_timeout(seer_ctx* ctx, int polls, void* stream) {
    if (!ctx) return SEER_ERR_INVALID_ARG;
    if (polls < 1 || polls > (1 << 20)) return fail(ctx, SEER_ERR_INVALID_ARG, "polls must lie in 1 .. 2^20");
    cudaError_t ce = cudaSetDevice(ctx->device);
    if (ce != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "cudaSetDevice: %s", cudaGetErrorString(ce));
    const WsLayout w = ws_layout(1, 0, 0, 0);
    debug_wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<unsigned int*>(ctx->ws), reinterpret_cast<unsigned long long*>(ctx->ws + w.tickets),
        reinterpret_cast<int*>(ctx->ws + w.sched), reinterpret_cast<int*>(ctx->ws + w.steal), (unsigned int)polls);
    ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "launch: %s", cudaGetErrorString(ce));
    ctx->launches += 1;
    return SEER_OK;
}

seer_status seer_get_device_status(seer_ctx* ctx, void* stream) {
    if (!ctx) return SEER_ERR_INVALID_ARG;
    cudaSetDevice(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, ctx->ws, sizeof word, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ws, 0, sizeof word, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "status read: %s", cudaGetErrorString(e));
    if (word & DEV_TIMEOUT) {
        // a CTA that gave up may have left tickets or scheduler counters behind: clear them
        const size_t fixed = ws_layout(1, 0, 0, 0).scratch;
        cudaMemsetAsync(ctx->ws + kStatusBytes, 0, (ctx->ws_bytes < fixed ? ctx->ws_bytes : fixed) - kStatusBytes, s);
        cudaStreamSynchronize(s);
        return fail(ctx, SEER_ERR_TIMEOUT, "a device-side wait gave up; results of that call are invalid");
    }
    if (word & DEV_BAD_INDEX) return fail(ctx, SEER_ERR_BAD_INDEX, "out-of-range block index or page id skipped");
    return SEER_OK;
}

size_t seer_workspace_bytes(const seer_shape* shape, int max_blocks, int d_gate) {
    if (!shape || shape->batch <= 0 || shape->num_kv_heads <= 0) return 0;
    const int U = shape->batch * shape->num_kv_heads;
    return ws_layout(U, decode_max_intervals(kMaxGridCtas) + U, d_gate, max_blocks, 2).total;   // (enough for every call; more lets the 17-to-64-row decode use more dynamic chunks)
}

seer_status seer_dense_decode(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv, const void* q, void* out,
                              float* lse, void* stream) {
    return decode_common(ctx, shape, kv, q, 1, nullptr, nullptr, 0, false, out, lse, stream);
}

seer_status seer_sparse_decode(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv, const void* q,
                               const int32_t* block_idx, const int32_t* block_cnt, int max_sel, void* out,
                               float* lse, void* stream) {
    return decode_common(ctx, shape, kv, q, 1, block_idx, block_cnt, max_sel, true, out, lse, stream);
}

seer_status seer_sparse_decode_multi(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv, const void* q,
                                     int q_len, const int32_t* block_idx, const int32_t* block_cnt, int max_sel,
                                     void* out, float* lse, void* stream) {
    return decode_common(ctx, shape, kv, q, q_len, block_idx, block_cnt, max_sel, true, out, lse, stream);
}

seer_status seer_dense_decode_multi(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv, const void* q,
                                    int q_len, void* out, float* lse, void* stream) {
    return decode_common(ctx, shape, kv, q, q_len, nullptr, nullptr, 0, false, out, lse, stream);
}

static seer_status gate_select_common(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate,
                                      const int32_t* seq_lens, const void* q_nope, const float* scores_in,
                                      int token_budget, int threshold_mode, float threshold, int32_t* block_idx,
                                      int32_t* block_cnt, int max_sel, float* scores_out, void* stream,
                                      int q_len = 1) {
    if (!ctx) return SEER_ERR_INVALID_ARG;
    seer_status st = check_shape(ctx, shape);
    if (st != SEER_OK) return st;
    if (!gate || !seq_lens || !block_idx || !block_cnt)
        return fail(ctx, SEER_ERR_INVALID_ARG, "NULL pointer among gate/seq_lens/block_idx/block_cnt");
    if (max_sel <= 0 || gate->max_blocks <= 0) return fail(ctx, SEER_ERR_INVALID_ARG, "max_sel and max_blocks must be positive");
    if (token_budget < 0) return fail(ctx, SEER_ERR_INVALID_ARG, "token_budget is negative");
    if (q_len < 1 || q_len > 8) return fail(ctx, SEER_ERR_UNSUPPORTED, "q_len %d (supported 1..8)", q_len);
    if (!scores_in) {
        if (!q_nope || !gate->w_q || !gate->kcomp)
            return fail(ctx, SEER_ERR_INVALID_ARG, "q_nope, w_q and kcomp are needed when scores_in is NULL");
        if (gate->d_gate != 64 && gate->d_gate != 128 && gate->d_gate != 256)
            return fail(ctx, SEER_ERR_UNSUPPORTED, "d_gate %d (supported: 64, 128, 256)", gate->d_gate);
        if (!aligned16(q_nope) || !aligned16(gate->w_q) || !aligned16(gate->kcomp))
            return fail(ctx, SEER_ERR_INVALID_ARG, "q_nope, w_q and kcomp must be 16-byte aligned");
        if (!(gate->rope_theta > 0.f)) return fail(ctx, SEER_ERR_INVALID_ARG, "rope_theta must be positive");
    }
    const int U = shape->batch * shape->num_kv_heads;
    const WsLayout w = ws_layout(U, 0, scores_in ? 0 : gate->d_gate, scores_in ? 0 : gate->max_blocks);
    if (w.total > ctx->ws_bytes)
        return fail(ctx, SEER_ERR_WORKSPACE, "workspace %zu bytes, call needs %zu", ctx->ws_bytes, w.total);
    cudaError_t ce = cudaSetDevice(ctx->device);
    if (ce != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "cudaSetDevice: %s", cudaGetErrorString(ce));

    GateParams p;
    memset(&p, 0, sizeof p);
    p.q_nope = static_cast<const __nv_bfloat16*>(q_nope);
    p.w_q = static_cast<const __nv_bfloat16*>(gate->w_q);
    p.kcomp = static_cast<const __nv_bfloat16*>(gate->kcomp);
    p.seq_lens = seq_lens;
    p.scores_in = scores_in;
    p.scores = scores_out ? scores_out : reinterpret_cast<float*>(ctx->ws + w.scores);
    p.scores_user = scores_out;
    p.q_gate = reinterpret_cast<float*>(ctx->ws + w.q_gate);
    p.block_idx = block_idx;
    p.block_cnt = block_cnt;
    p.batch = shape->batch;
    p.num_q_heads = shape->num_q_heads;
    p.num_kv_heads = shape->num_kv_heads;
    p.group = shape->num_q_heads / shape->num_kv_heads;
    p.block_size = shape->block_size;
    p.d_gate = gate->d_gate;
    p.max_blocks = gate->max_blocks;
    p.max_sel = max_sel;
    p.token_budget = token_budget;
    p.q_len = q_len;
    p.threshold_mode = threshold_mode;
    p.threshold = threshold;
    p.status = reinterpret_cast<unsigned int*>(ctx->ws);
    p.tickets = reinterpret_cast<int*>(ctx->ws + w.gate_tickets);
    if (ctx->list_gen != 0) {
        p.list_flags = reinterpret_cast<int*>(ctx->ws + w.list_flags);
        p.list_gen = ctx->list_gen;
    }
#ifdef SEER_GATE_TRACE
    p.status = reinterpret_cast<unsigned int*>(ctx->ws + (ctx->ws_bytes - (size_t)(1 << 19)));
#endif
    if (!scores_in) fill_inv_freq(p.inv_freq, gate->d_gate, gate->rope_theta);
    int launched = 0;
    ce = launch_gate_select(p, static_cast<cudaStream_t>(stream), &launched);
    ctx->launches += launched;
    if (ce != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "gate launch: %s", cudaGetErrorString(ce));
    return SEER_OK;
}

seer_status seer_gate_select(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate, const int32_t* seq_lens,
                             const void* q_nope, const float* scores_in, int token_budget, int32_t* block_idx,
                             int32_t* block_cnt, int max_sel, float* scores_out, void* stream) {
    return gate_select_common(ctx, shape, gate, seq_lens, q_nope, scores_in, token_budget, 0, 0.f, block_idx, block_cnt,
                              max_sel, scores_out, stream);
}

seer_status seer_gate_select_multi(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate,
                                   const int32_t* seq_lens, const void* q_nope, const float* scores_in, int q_len,
                                   int token_budget, int32_t* block_idx, int32_t* block_cnt, int max_sel,
                                   float* scores_out, void* stream) {
    return gate_select_common(ctx, shape, gate, seq_lens, q_nope, scores_in, token_budget, 0, 0.f, block_idx, block_cnt,
                              max_sel, scores_out, stream, q_len);
}

seer_status seer_gate_select_threshold(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate,
                                       const int32_t* seq_lens, const void* q_nope, const float* scores_in,
                                       float threshold, int32_t* block_idx, int32_t* block_cnt, int max_sel,
                                       float* scores_out, void* stream) {
    if (ctx && !(threshold >= 0.f && threshold <= 1.f))
        return fail(ctx, SEER_ERR_INVALID_ARG, "threshold must lie in [0, 1] (it is compared with a softmax probability)");
    return gate_select_common(ctx, shape, gate, seq_lens, q_nope, scores_in, 0, 1, threshold, block_idx, block_cnt, max_sel,
                              scores_out, stream);
}

static seer_status kcomp_append_common(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate, const int32_t* seq_lens,
                                       const void* k_nope, int64_t stride_batch, int64_t stride_head, int64_t stride_token,
                                       int rows_block_local, int first_block, int num_blocks, int wait_at_end, void* stream) {
    if (!ctx) return SEER_ERR_INVALID_ARG;
    seer_status st = check_shape(ctx, shape);
    if (st != SEER_OK) return st;
    if (!gate || !seq_lens || !k_nope || !gate->w_k || !gate->kcomp)
        return fail(ctx, SEER_ERR_INVALID_ARG, "NULL pointer among gate/seq_lens/k_nope/w_k/kcomp");
    if (gate->d_gate != 64 && gate->d_gate != 128 && gate->d_gate != 256)
        return fail(ctx, SEER_ERR_UNSUPPORTED, "d_gate %d (supported: 64, 128, 256)", gate->d_gate);
    if (gate->max_blocks <= 0) return fail(ctx, SEER_ERR_INVALID_ARG, "max_blocks must be positive");
    if (!(gate->rope_theta > 0.f)) return fail(ctx, SEER_ERR_INVALID_ARG, "rope_theta must be positive");
    if (!aligned16(k_nope) || !aligned16(gate->w_k) || !aligned16(gate->kcomp))
        return fail(ctx, SEER_ERR_INVALID_ARG, "k_nope, w_k and kcomp must be 16-byte aligned");
    if (stride_batch % 8 || stride_head % 8 || stride_token % 8 || stride_token < kHeadDim || stride_batch < 0 ||
        stride_head < 0)
        return fail(ctx, SEER_ERR_INVALID_ARG, "k_nope strides must be multiples of 8 elements");
    if (first_block < -8) return fail(ctx, SEER_ERR_INVALID_ARG, "first_block must be >= -8");
    if (first_block >= 0 && num_blocks < 0) return fail(ctx, SEER_ERR_INVALID_ARG, "num_blocks is negative");
    if (first_block >= 0 && rows_block_local && num_blocks > 1)
        return fail(ctx, SEER_ERR_INVALID_ARG, "a block-local buffer holds one block only");
    cudaError_t ce = cudaSetDevice(ctx->device);
    if (ce != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "cudaSetDevice: %s", cudaGetErrorString(ce));

    KcompParams p;
    memset(&p, 0, sizeof p);
    p.k_nope = static_cast<const __nv_bfloat16*>(k_nope);
    p.w_k = static_cast<const __nv_bfloat16*>(gate->w_k);
    p.kcomp = static_cast<__nv_bfloat16*>(gate->kcomp);
    p.seq_lens = seq_lens;
    p.stride_batch = stride_batch;
    p.stride_head = stride_head;
    p.stride_token = stride_token;
    p.rows_block_local = rows_block_local;
    p.first_block = first_block;
    p.num_blocks = num_blocks;
    p.batch = shape->batch;
    p.num_kv_heads = shape->num_kv_heads;
    p.block_size = shape->block_size;
    p.d_gate = gate->d_gate;
    p.max_blocks = gate->max_blocks;
    p.wait_at_end = wait_at_end;
    p.sm_count = ctx->num_sms;
    p.status = reinterpret_cast<unsigned int*>(ctx->ws);
#ifdef SEER_DECODE_TRACE
    p.trace = reinterpret_cast<unsigned long long*>(ctx->ws + (ctx->ws_bytes - (size_t)(1 << 20)));
#endif
    fill_inv_freq(p.inv_freq, gate->d_gate, gate->rope_theta);
    const CUtensorMap* map_k = nullptr;
    if (kcomp_bulk_streams(p)) {
        // (channel, token row, head, sequence); the row extent is the last row the build may touch
        const uint64_t dims[4] = {(uint64_t)kHeadDim, (uint64_t)(first_block + num_blocks) * (uint64_t)shape->block_size,
                                  (uint64_t)shape->num_kv_heads, (uint64_t)shape->batch};
        const uint64_t strides[3] = {(uint64_t)stride_token * 2, (uint64_t)stride_head * 2, (uint64_t)stride_batch * 2};
        st = get_map(ctx, k_nope, dims, strides, kKcompStageRows, &map_k);
        if (st != SEER_OK) return st;
    }
    int launched = 0;
    ce = launch_kcomp_append(p, map_k, static_cast<cudaStream_t>(stream), &launched);
    ctx->launches += launched;
    if (ce != cudaSuccess) return fail(ctx, SEER_ERR_CUDA, "kcomp launch: %s", cudaGetErrorString(ce));
    return SEER_OK;
}

seer_status seer_gate_select_threshold_multi(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate,
                                             const int32_t* seq_lens, const void* q_nope, const float* scores_in,
                                             int q_len, float threshold, int32_t* block_idx, int32_t* block_cnt,
                                             int max_sel, float* scores_out, void* stream) {
    if (ctx && !(threshold >= 0.f && threshold <= 1.f))
        return fail(ctx, SEER_ERR_INVALID_ARG, "threshold must lie in [0, 1] (it is compared with a softmax probability)");
    return gate_select_common(ctx, shape, gate, seq_lens, q_nope, scores_in, 0, 1, threshold, block_idx, block_cnt, max_sel,
                              scores_out, stream, q_len);
}

seer_status seer_kcomp_append(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate, const int32_t* seq_lens,
                              const void* k_nope, int64_t stride_batch, int64_t stride_head, int64_t stride_token,
                              int rows_block_local, int first_block, int num_blocks, void* stream) {
    return kcomp_append_common(ctx, shape, gate, seq_lens, k_nope, stride_batch, stride_head, stride_token,
                               rows_block_local, first_block, num_blocks, 0, stream);
}

seer_status seer_decode_step(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv, const seer_gate* gate,
                             const void* q, const void* q_nope, const void* k_nope, int64_t k_nope_stride_batch,
                             int64_t k_nope_stride_head, int64_t k_nope_stride_token, int k_nope_rows_block_local,
                             int token_budget, int32_t* block_idx, int32_t* block_cnt, int max_sel, void* out,
                             float* lse, void* stream) {
    if (!ctx) return SEER_ERR_INVALID_ARG;
    if (!kv || !kv->seq_lens) return fail(ctx, SEER_ERR_INVALID_ARG, "kv or kv->seq_lens is NULL");
    // The block that has just filled is the sequence's last block, which the gate always selects without
    // scoring it (Sec. 3.2): its compressed key is first needed in the next step.  The append is therefore
    // the step's last launch and does its work under the tail of the attention kernel.
    // With the token budget every list has min(budget in blocks, blocks of the sequence) entries (as long as the
    // compressed-key cache covers the longest sequence): the attention kernel then counts its tiles from the
    // lengths, before the gate has finished, and waits, unit by unit, for the mark the gate kernel leaves when a
    // unit's list is written.
    if (!shape || !gate) return fail(ctx, SEER_ERR_INVALID_ARG, "shape or gate is NULL");
    const int k_blocks = token_budget / shape->block_size > 1 ? token_budget / shape->block_size : 1;
    const bool covered = (long long)gate->max_blocks * shape->block_size >= (long long)kv->max_seq_len;
    if (covered && ctx->use_list_flags) {
        ctx->list_gen_last = ctx->list_gen_last >= 0x7ffffff0 ? 1 : ctx->list_gen_last + 1;
        ctx->list_gen = ctx->list_gen_last;
    }
    seer_status st = seer_gate_select(ctx, shape, gate, kv->seq_lens, q_nope, nullptr, token_budget, block_idx, block_cnt,
                                      max_sel, nullptr, stream);
    if (st != SEER_OK) {
        ctx->list_gen = 0;
        return st;
    }
    ctx->sel_from_lens = covered ? (k_blocks < max_sel ? k_blocks : max_sel) : 0;
    st = seer_sparse_decode(ctx, shape, kv, q, block_idx, block_cnt, max_sel, out, lse, stream);
    ctx->sel_from_lens = 0;
    ctx->list_gen = 0;
    if (st != SEER_OK || !k_nope) return st;
    return kcomp_append_common(ctx, shape, gate, kv->seq_lens, k_nope, k_nope_stride_batch, k_nope_stride_head,
                               k_nope_stride_token, k_nope_rows_block_local, -1, 1, 1, stream);
}

seer_status seer_decode_step_multi(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv, const seer_gate* gate,
                                   const void* q, const void* q_nope, int q_len, const void* k_nope,
                                   int64_t k_nope_stride_batch, int64_t k_nope_stride_head, int64_t k_nope_stride_token,
                                   int k_nope_rows_block_local, int token_budget, int32_t* block_idx,
                                   int32_t* block_cnt, int max_sel, void* out, float* lse, void* stream) {
    if (!ctx) return SEER_ERR_INVALID_ARG;
    if (!kv || !kv->seq_lens) return fail(ctx, SEER_ERR_INVALID_ARG, "kv or kv->seq_lens is NULL");
    if (q_len < 1 || q_len > 8) return fail(ctx, SEER_ERR_UNSUPPORTED, "q_len %d (supported 1..8)", q_len);
    // (the block that filled holds one of the query tokens, so it is among the blocks selected without a
    // score: as in seer_decode_step the append comes last)
    seer_status st = seer_gate_select_multi(ctx, shape, gate, kv->seq_lens, q_nope, nullptr, q_len, token_budget, block_idx,
                                            block_cnt, max_sel, nullptr, stream);
    if (st != SEER_OK) return st;
    st = seer_sparse_decode_multi(ctx, shape, kv, q, q_len, block_idx, block_cnt, max_sel, out, lse, stream);
    if (st != SEER_OK || !k_nope) return st;
    return kcomp_append_common(ctx, shape, gate, kv->seq_lens, k_nope, k_nope_stride_batch, k_nope_stride_head,
                               k_nope_stride_token, k_nope_rows_block_local, -q_len, 1, 1, stream);
}

}  // extern "C"
