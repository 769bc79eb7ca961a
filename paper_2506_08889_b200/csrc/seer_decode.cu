// Split-KV flash decoding for GQA on sm_100a: the block-sparse kernel of Sec. 3.3 and the
// dense kernel built from the same parts.
//
// Work decomposition.  A "unit" is one (sequence, KV head) pair; its work is the list of
// 64-token tiles of its selected blocks (sparse) or of its whole sequence (dense).  All
// units' tile lists are laid end to end (T tiles) and cut into one equal contiguous range per
// CTA.  The first three quarters of a range are its CTA's static share; the last quarter is
// cut into chunks of geometrically varying size (two tiles ... 1/8 of the range; see Schedule for
// their order).  The owner of a range claims its chunks from the front, so its work stays one
// contiguous run; a CTA that has finished its own range steals other ranges' chunks from the
// back.
// SMs that get less memory bandwidth than others thus shed work to faster ones and all finish
// together, while a unit is cut into few pieces.  Claims are single atomic adds on a per-range
// counter; nobody ever waits for another CTA.
//
// A piece is a maximal run of one unit's tiles that one CTA processes in one go.  A piece that
// covers its unit completely writes the final output.  Any other piece writes an un-normalised
// partial (o, max, sum), stamped with the launch's generation number, into the slot of the
// interval it starts in.  When a CTA has finished streaming it adds the tile counts of its pieces
// to their units' counters; whoever completes a unit's count merges that unit's partials
// (log-sum-exp combine over the valid slots among the unit's intervals), with all of its warps.
//
// Inside a CTA: one producer warp walks the intervals, turns each tile into TMA box loads
// (K and V, 2 x 64x64 bf16 boxes each, 128-byte swizzle) into a ring of shared-memory
// stages, and passes per-tile metadata beside the data.  Four consumer warps each own 16
// of a tile's 64 tokens and keep private online-softmax state (running max, sum, and the
// 128 x 8 output accumulator), so they never synchronise with each other inside the loop:
//     S^T (16 tok x 8 heads) = K_slice (16 x 128) . Q^T (128 x 8)      mma.sync m16n8k16
//     P^T -> bf16, transposed in registers (movmatrix) into the B operand
//     O^T (128 x 8)        += V_slice^T (128 x 16) . P^T (16 x 8)       mma.sync m16n8k16
// The g <= 8 query heads of the group sit on the MMA's N = 8 side, tokens on M.
//
// Template variants.  NT = 2 puts up to 16 rows on the N side (two N-tiles per warp): several query
// tokens per sequence, row = (token, head), each row cut off causally at its own position.  SMALL
// gathers four or two listed blocks of 16 or 32 tokens into one 64-token tile (one TMA box per
// block, one valid-token count per block); blocks of 64 or 128 tokens are one or two tiles.
#include "seer_device.cuh"
#include "seer_internal.h"

namespace seer {

namespace {

constexpr int kStages = 3;
constexpr int kConsumerWarps = 4;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;
constexpr int kHalfTileBytes = kTileTokens * 128;          // 64 rows x 128 B (64 bf16 channels)
constexpr int kTileBytes = 2 * kHalfTileBytes;             // one K or V tile: 16 KiB
constexpr int kStageBytes = 2 * kTileBytes;                // K + V
constexpr int kMergeStride = 132;                          // floats per head row (bank spread)
constexpr int kMaxPieces = 32;                             // partial pieces a CTA can hold back to its end
constexpr int kListInts = kStageBytes / 4 - 64;              // slot numbers that fit in one stage buffer (less 64 counts)
constexpr int kMaxSteals = 14;                             // chunks a CTA may take from other ranges
constexpr int kFewTilesPerCta = 16;                        // up to this many tiles per CTA the number of ranges is chosen with care
constexpr int kWideTiles = 8;                              // N-tile count that stands for the rows-on-M variant (up to 64 rows)
// The rows-on-M variant on the fifth-generation tensor cores (TC): one CTA per SM, a deeper ring, an extra
// warp that issues the MMAs; S, P, O and the unit's queries live in tensor memory.
constexpr int kTcTilesCode = 16;                           // what the host passes as n_tiles to ask for it
constexpr int kTcStages = 7;                               // V buffers (16 KiB each) = tiles between landing and product
constexpr int kTcKStages = 5;                              // K buffers (16 KiB each): a K tile is free once its scores are computed
constexpr int kTcThreads = kThreads + 32;
constexpr int kTcRows = 128;                               // M of the MMAs (rows past the unit's are padding: zero, or never read)
constexpr int kTcSBufs = 3;                                // S/P buffers: scores of up to three tiles ahead of their products
constexpr int kTcOCol = 64 * kTcSBufs, kTcQCol = kTcOCol + 128;   // tensor-memory columns of O and of Q
constexpr int kTcCols = 512;                               // S/P 3 x 64, O 128, Q 64 = 384 columns, as a power of two
constexpr int kAheadMaxChunk = 8;                          // own chunks up to this size are claimed ahead
constexpr int kAheadTiles = 3;                             // tiles left to issue when the next interval's claim is made
constexpr int kSmemUnits = 128;                            // units whose tile-count prefix sums fit in shared memory
constexpr int kMinChunk = 2;                               // smallest dynamic chunk, in tiles
constexpr int kMinStaticTilesPerCta = 8;                   // below this everything is static

struct StageMeta {
    int nvalid;        // cached tokens from the tile's first row on, capped at 64 + 7 (0 = nothing was loaded); -1 = end of
                       // stream.  Blocks of 16 or 32 tokens: one such count per gathered block, 8 bits each (capped at b + 7)
    int unit;          // (sequence, KV head) index
    int flags;         // bit 0: first tile of a piece
    int unit_first;    // global index of the unit's first tile
    int unit_tiles;    // tiles of the unit
    int interval;      // interval this tile belongs to
};

// A partial this CTA wrote (unit, tiles, first candidate slot of the unit, number of candidate slots,
// tiles of the unit); after the stream the same records list the units this CTA has to combine
// (unit, -, first_slot, n_slots, mask of valid slots or 0 if unknown).
struct Piece {
    int unit, tiles, unit_first, unit_tiles, extra;
};

// Geometry of the intervals, identical in every CTA (derived from T and gridDim.x).  Range c = [a, b)
// is cut into its static share [a, b - off[1]) and R chunks [b - off[j], b - off[j+1]), j = 1..R
// (off[R+1] = 0).  The chunks cover the last quarter of the range and halve towards its end (1/8, 1/16,
// ... of the range, down to kMinChunk tiles), except that none is longer than 8 tiles (16 from ranges of
// 512 tiles on, 32 from 1024 on, ...): longer ones are cut up.  The owner, coming from the front, meets the bigger
// chunks, thieves take the small ones at the back first, and no chunk is so big that a slow owner who
// has just claimed it holds everybody up.
struct Schedule {
    int T, G;                      // tiles, ranges (G <= T)
    int R;                         // dynamic chunks per range (0: everything is static)
    int q, r;                      // T = q * G + r: ranges of q tiles, the first r of them one tile longer
    int off[kMaxRounds + 2];       // off[j]: tiles from the start of chunk j to the end of its range
};

// What only one kind of variant needs: the cross-warp merge scratch of the mma.sync variants, or the barriers of
// the tensor-memory variant.
template <bool TC>
struct VariantPart {
    float merge_o[kConsumerWarps - 1][kMaxGroup][kMergeStride];   // warps 1..3 -> warp 0
    float merge_ml[kConsumerWarps - 1][2][kMaxGroup];
};
template <>
struct VariantPart<true> {
    uint64_t bar_s[kTcSBufs];        // S of a tile (buffer = tile number mod kTcSBufs) is complete (the MMA warp's commit)
    uint64_t bar_p[kTcSBufs];        // P of such a tile is written (one arrival per row warp with real rows)
    uint64_t bar_o[kTcSBufs];        // O includes such a tile's product (commit)
    uint64_t bar_q;                  // the queries of a piece's unit are in tensor memory (one arrival per row warp with real rows)
    uint64_t tmem_done;              // the row warps have made their last tensor-memory access
    uint64_t empty_k[kTcKStages];    // a K buffer's scores have been computed (commit)
    uint32_t tmem_base;
};

template <bool TC>
struct __align__(1024) SmemT {
    static constexpr int kS = TC ? kTcStages : kStages;
    // The K/V ring.  The tensor-memory variant cuts the same memory differently: kTcStages V buffers, then
    // kTcKStages K buffers (16 KiB each).
    static constexpr int kBufs = TC ? (kTcStages + kTcKStages) / 2 : kStages;
    unsigned char stage[kBufs][kStageBytes];
    uint64_t full[kS];
    uint64_t empty[kS];
    uint64_t merge_bar[2];           // [0]: scratch filled (3 arrivals), [1]: scratch free again / end sync
    uint64_t end_bar;                // all consumer warps: streams over, the list of combines is final
    uint64_t list_bar;               // all consumer warps: the lists of valid slots are written
    uint64_t land_bar;               // bulk copies of partials into the landing area have arrived
    volatile int issued;             // tiles whose metadata the producer has written so far
    volatile int first_unit;         // unit of the CTA's first tile (-1: none yet known, -2: not yet decided)
    int upfx[kSmemUnits + 1];        // prefix sums of the units' tile counts (when there are at most kSmemUnits units)
    StageMeta meta[kS];
    Schedule sched;
    Piece pieces[kMaxPieces];
    int pieces_n;
    VariantPart<TC> v;
};
static_assert((kTcStages + kTcKStages) % 2 == 0, "the K and V buffers fill whole stage buffers");
using Smem = SmemT<false>;
static_assert(sizeof(SmemT<true>) + 1024 <= 227 * 1024, "the tensor-memory variant's shared memory");

// two CTAs per SM: 2 * (sizeof(Smem) + 1 KiB alignment slack + 1 KiB reserved by the system) must
// fit in the SM's 228 KiB
static_assert(sizeof(Smem) + 1024 <= 113 * 1024, "decode kernel no longer fits two CTAs per SM");

#ifdef SEER_DECODE_TRACE
// diagnostic builds: per CTA, slots 0..15 are named stamps, slots 16.. the arrival time of every tile
constexpr int kTraceSlots = 128;
__device__ __forceinline__ void trace_stamp(const DecodeParams& p, int slot) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    p.trace[(size_t)blockIdx.x * kTraceSlots + slot] = t;
}
#define SEER_STAMP(slot) trace_stamp(p, slot)
#else
#define SEER_STAMP(slot) ((void)0)
#endif

// Sequence of unit u (u / num_kv_heads by a multiplication: kvh_magic = ceil(2^32 / num_kv_heads), exact
// for the 16-bit unit numbers the library takes; 0 stands for one KV head).
__device__ __forceinline__ int unit_seq(const DecodeParams& p, int u) {
    return p.kvh_magic ? (int)__umulhi((unsigned int)u, p.kvh_magic) : u;
}

template <bool SPARSE, bool SMALL = false>
__device__ __forceinline__ int tiles_of(const DecodeParams& p, int u) {
    const int L = p.seq_lens[unit_seq(p, u)];
    if (SPARSE) {
        int c;
        if (p.sel_from_lens > 0) {
            c = min(p.sel_from_lens, (L + p.block_size - 1) >> p.bs_shift);     // (the lists are not final yet)
        } else {
            c = p.block_cnt ? p.block_cnt[u] : p.max_sel;     // not behind the test on L: both loads in flight
        }
        c = max(0, min(c, p.max_sel));
        return L <= 0 ? 0 : (SMALL ? (c + p.blocks_per_tile - 1) >> p.bpt_shift : c << p.tpb_shift);
    } else {
        if (L <= 0) return 0;
        int t = (L + kTileTokens - 1) / kTileTokens;
        return min(t, p.max_blocks_cap);
    }
}

// T tiles are cut into G contiguous ranges of q = T / G tiles, the first r = T % G of them one tile
// longer: range c begins at c*q + min(c, r).
__device__ __forceinline__ int range_begin(const Schedule& s, int c) { return c * s.q + min(c, s.r); }
__device__ __forceinline__ int range_of(const Schedule& s, int t) {
    const int long_part = s.r * (s.q + 1);
    return t < long_part ? (int)((unsigned int)t / (unsigned int)(s.q + 1))
                         : s.r + (int)((unsigned int)(t - long_part) / (unsigned int)s.q);
}

// Run by a whole warp: the scalar fields come out in every lane's copy `s`, the table is written to
// `shared`, where all of the schedule is also left for the other warps.  Lane k takes level k of the
// tail, [b - (q/4 >> k), b - (q/4 >> (k+1))), and cuts it into pieces of `cap` tiles (a power of two)
// counted from its back end, the front piece taking the remainder.
__device__ __forceinline__ void build_schedule(Schedule& s, Schedule& shared, int T, int grid, int pool_div, int max_rounds,
                                               int lane) {
    s.T = T;
    s.G = max(1, min(grid, T));
    const int q = (int)((unsigned int)T / (unsigned int)s.G);   // shortest range (>= 1 whenever T > 0)
    s.q = q;
    s.r = T - q * s.G;
    int R = 0;
    if (pool_div > 0 && q >= kMinStaticTilesPerCta) {
        const int tail = pool_div == 4 ? q >> 2 : q / pool_div;
        // (with one piece per level there are at most max_rounds pieces, so the loop ends at the latest
        // when cap exceeds the tail)
                for (int cap_shift = 3 + max(0, 23 - __clz(q)); cap_shift < 31; ++cap_shift) {      // cap = 8, or about q/32 .. q/64
            // level k = [b - prev, b - nxt): halves, down to kMinChunk tiles; the last level takes the rest
            int prev = lane < max_rounds ? tail >> lane : 0;
            if (lane > 0 && prev < kMinChunk) prev = 0;
            int nxt = prev >> 1;
            if (nxt < kMinChunk || lane == max_rounds - 1) nxt = 0;
            const int size = prev - nxt;                    // (0 for the levels past the last)
            const int parts = (size + (1 << cap_shift) - 1) >> cap_shift;
            int incl = parts;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            R = __shfl_sync(0xffffffffu, incl, 31);
            if (R > max_rounds) { R = 0; continue; }
            // piece i of the level (front to back) starts prev tiles before the range's end for i = 0,
            // nxt + (parts - i) * cap for the others
            for (int i = 0; i < parts; ++i) shared.off[incl - parts + 1 + i] = i == 0 ? prev : nxt + ((parts - i) << cap_shift);
            break;
        }
    }
    s.R = R;
    if (lane == 0) {
        shared.off[R + 1] = 0;
        shared.T = s.T; shared.G = s.G; shared.R = R; shared.q = q; shared.r = s.r;
    }
    __syncwarp();
}

// Interval j (0 = static share, 1..R = chunks, front to back) of range c.
// (s: the scalar fields, possibly a register copy; off: the table in shared memory)
__device__ __forceinline__ void interval_range(const Schedule& s, const int* off, int c, int j, int* begin, int* end) {
    const int a = range_begin(s, c), b = range_begin(s, c + 1);
    if (s.R == 0) { *begin = a; *end = b; return; }
    *begin = j == 0 ? a : b - off[j];
    *end = b - off[j + 1];
}

// Number (c * (R+1) + j, increasing with the tile position) of the interval that holds tile t.
__device__ __forceinline__ int interval_of(const Schedule& s, int t) {
    const int c = range_of(s, t);
    if (s.R == 0) return c;
    const int d = range_begin(s, c + 1) - t;        // tiles from t to the end of its range (>= 1)
    int j = 0;
    while (j < s.R && d <= s.off[j + 1]) ++j;
    return c * (s.R + 1) + j;
}

// Output row of row r on a unit's MMA N side: query token t_base + r / group, head r % group of
// the KV head's group; rows of q, out and lse are laid out [sequence][token][query head].
__device__ __forceinline__ size_t unit_row(const DecodeParams& p, int u, int r) {
    const int i = unit_seq(p, u), h = u - i * p.num_kv_heads;
    const int tl = (r * p.group_magic) >> 16, gi = r - tl * p.group;      // r / group for r < 16
    return ((size_t)i * p.q_len + p.t_base + tl) * p.num_q_heads + (size_t)h * p.group + gi;
}

__device__ __forceinline__ void write_zero_unit(const DecodeParams& p, int u) {
    for (int r = 0; r < p.rows; ++r) {
        const size_t row = unit_row(p, u, r);
        for (int c = 0; c < kHeadDim; ++c) p.out[row * kHeadDim + c] = __float2bfloat16(0.f);
        if (p.lse) p.lse[row] = -INFINITY;
    }
}

// floats per slot in part_ml for a kernel with one N-tile: [0..7] max, [8..15] sum, [16] generation;
// with NT N-tiles: [0..8NT) max, [8NT..16NT) sum, [16NT] generation, 32*NT floats in all
constexpr int kMlStride = 32;

// Log-sum-exp combine of one unit's partials by the CTA's consumer threads.  Thread t takes rows
// t/16 + 8*nt, channels 8*(t%16) .. +7 of every partial.
template <int NT>
struct MergeState {
    float M[NT], lsum[NT], acc[NT][8];
};
template <int NT>
__device__ __forceinline__ void merge_init(MergeState<NT>& st) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        st.M[nt] = -INFINITY;
        st.lsum[nt] = 0.f;
#pragma unroll
        for (int x = 0; x < 8; ++x) st.acc[nt][x] = 0.f;
    }
}
// Adds up to kDirect partials straight from global memory: every load (of one N-tile's rows) is
// issued before any arithmetic, so the whole batch costs one round trip to L2 per N-tile (the
// cheapest way for a few partials).
constexpr int kDirect = 8;
template <int NT>
__device__ __forceinline__ void merge_accumulate_direct(const DecodeParams& p, MergeState<NT>& st,
                                                        const int (&slots)[kDirect], int n, int t) {
    const int d0 = 8 * (t & 15);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int hh = (t >> 4) + 8 * nt;
        float ms[kDirect], ls[kDirect];
        float4 va[kDirect], vb[kDirect];
#pragma unroll
        for (int k = 0; k < kDirect; ++k) {
            const size_t sl = (size_t)slots[k];            // (entries from n on repeat a valid slot)
            const float* pm = p.part_ml + sl * (kMlStride * NT);
            const float4* qo = reinterpret_cast<const float4*>(p.part_o + sl * (8 * NT * kHeadDim) + hh * kHeadDim + d0);
            ms[k] = __ldcg(pm + hh);
            ls[k] = __ldcg(pm + 8 * NT + hh);
            va[k] = __ldcg(qo);
            vb[k] = __ldcg(qo + 1);
        }
        float Mr = st.M[nt];
#pragma unroll
        for (int k = 0; k < kDirect; ++k) Mr = fmaxf(Mr, k < n ? ms[k] : -INFINITY);
        if (Mr == -INFINITY) continue;
        const float fo = (st.M[nt] == -INFINITY) ? 0.f : fast_exp2(st.M[nt] - Mr);
        st.M[nt] = Mr;
        st.lsum[nt] *= fo;
#pragma unroll
        for (int x = 0; x < 8; ++x) st.acc[nt][x] *= fo;
#pragma unroll
        for (int k = 0; k < kDirect; ++k) {
            const float fn = (k < n && ms[k] != -INFINITY) ? fast_exp2(ms[k] - Mr) : 0.f;
            st.lsum[nt] = fmaf(ls[k], fn, st.lsum[nt]);
            st.acc[nt][0] = fmaf(va[k].x, fn, st.acc[nt][0]); st.acc[nt][1] = fmaf(va[k].y, fn, st.acc[nt][1]);
            st.acc[nt][2] = fmaf(va[k].z, fn, st.acc[nt][2]); st.acc[nt][3] = fmaf(va[k].w, fn, st.acc[nt][3]);
            st.acc[nt][4] = fmaf(vb[k].x, fn, st.acc[nt][4]); st.acc[nt][5] = fmaf(vb[k].y, fn, st.acc[nt][5]);
            st.acc[nt][6] = fmaf(vb[k].z, fn, st.acc[nt][6]); st.acc[nt][7] = fmaf(vb[k].w, fn, st.acc[nt][7]);
        }
    }
}

// Adds the partials that have been staged in shared memory: land_o + k * o_stride holds the
// rows x 128 floats of partial k, land_ml + k * 32 * NT its (max, sum, stamp) record.
template <int NT>
__device__ __forceinline__ void merge_accumulate_staged(MergeState<NT>& st, const float* land_o, int o_stride,
                                                        const float* land_ml, int m, int rows, int t) {
    const int d0 = 8 * (t & 15);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int hh = (t >> 4) + 8 * nt;
        if (hh >= rows) continue;
        // the round's maximum first, so that the sum below is a chain of independent multiply-adds
        float Mr = st.M[nt];
        for (int k = 0; k < m; ++k) Mr = fmaxf(Mr, land_ml[k * (kMlStride * NT) + hh]);
        if (Mr == -INFINITY) continue;
        const float fo = (st.M[nt] == -INFINITY) ? 0.f : fast_exp2(st.M[nt] - Mr);
        st.M[nt] = Mr;
        st.lsum[nt] *= fo;
#pragma unroll
        for (int x = 0; x < 8; ++x) st.acc[nt][x] *= fo;
#pragma unroll 4
        for (int k = 0; k < m; ++k) {
            const float ms = land_ml[k * (kMlStride * NT) + hh];
            const float fn = (ms == -INFINITY) ? 0.f : fast_exp2(ms - Mr);
            const float4 va = *reinterpret_cast<const float4*>(land_o + k * o_stride + hh * kHeadDim + d0);
            const float4 vb = *reinterpret_cast<const float4*>(land_o + k * o_stride + hh * kHeadDim + d0 + 4);
            st.lsum[nt] = fmaf(land_ml[k * (kMlStride * NT) + 8 * NT + hh], fn, st.lsum[nt]);
            st.acc[nt][0] = fmaf(va.x, fn, st.acc[nt][0]); st.acc[nt][1] = fmaf(va.y, fn, st.acc[nt][1]);
            st.acc[nt][2] = fmaf(va.z, fn, st.acc[nt][2]); st.acc[nt][3] = fmaf(va.w, fn, st.acc[nt][3]);
            st.acc[nt][4] = fmaf(vb.x, fn, st.acc[nt][4]); st.acc[nt][5] = fmaf(vb.y, fn, st.acc[nt][5]);
            st.acc[nt][6] = fmaf(vb.z, fn, st.acc[nt][6]); st.acc[nt][7] = fmaf(vb.w, fn, st.acc[nt][7]);
        }
    }
}
template <int NT>
__device__ __forceinline__ void merge_finalize(const DecodeParams& p, const MergeState<NT>& st, int u, int t) {
    const int d0 = 8 * (t & 15);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int hh = (t >> 4) + 8 * nt;
        if (hh >= p.rows) continue;
        const size_t row = unit_row(p, u, hh);
        const float inv = st.lsum[nt] > 0.f ? 1.f / st.lsum[nt] : 0.f;
        uint4 pk;
        pk.x = pack_bf16x2(st.acc[nt][0] * inv, st.acc[nt][1] * inv);
        pk.y = pack_bf16x2(st.acc[nt][2] * inv, st.acc[nt][3] * inv);
        pk.z = pack_bf16x2(st.acc[nt][4] * inv, st.acc[nt][5] * inv);
        pk.w = pack_bf16x2(st.acc[nt][6] * inv, st.acc[nt][7] * inv);
        *reinterpret_cast<uint4*>(p.out + row * kHeadDim + d0) = pk;
        if (p.lse && (t & 15) == 0)
            p.lse[row] = st.lsum[nt] > 0.f ? (st.M[nt] + log2f(st.lsum[nt])) * 0.6931471805599453f : -INFINITY;
    }
}
// One warp: the slots among [first, first + n_slots) that carry this launch's generation stamp,
// written to `list` in order; returns how many.
template <int NT>
__device__ __forceinline__ int scan_valid_slots(const DecodeParams& p, int first, int n_slots, int* list, int lane) {
    int n = 0;
    // four stamps per lane in flight: the scan costs one round trip per 128 candidate slots
    for (int s0 = 0; s0 < n_slots; s0 += 128) {
        unsigned int stamp[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int x = s0 + 32 * k + lane;
            stamp[k] = x < n_slots ? __float_as_uint(__ldcg(p.part_ml + (size_t)(first + x) * (kMlStride * NT) + 16 * NT))
                                   : ~p.generation;
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool ok = stamp[k] == p.generation;
            const unsigned m = __ballot_sync(0xffffffffu, ok);
            if (ok) list[n + __popc(m & ((1u << lane) - 1u))] = first + s0 + 32 * k + lane;
            n += __popc(m);
        }
    }
    return n;
}

template <bool SPARSE, bool PAGED, int NT, bool SMALL, bool TC = false>
__global__ void __launch_bounds__(TC ? kTcThreads : kThreads, TC ? 1 : 2)
decode_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
              const DecodeParams p) {
    static_assert(!TC || (NT == kWideTiles && !SMALL), "the tensor-memory variant is the rows-on-M variant");
    using SmemK = SmemT<TC>;
    constexpr int kS = SmemK::kS;    // stages of the K/V ring
    extern __shared__ unsigned char smem_raw[];
    SmemK& sm = *reinterpret_cast<SmemK*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int U = p.num_units;
    const int cta = blockIdx.x;

    if (tid == 0) {
        // row warps that hold real rows of the unit (tensor-memory variant: lane = row, 32 rows per warp)
        const int tc_row_warps = min(kConsumerWarps, (p.rows + 31) / 32);
        for (int s = 0; s < kS; ++s) {
            mbar_init(&sm.full[s], 1);
            // a stage is free once every consumer warp has arrived; tensor-memory variant: once the MMAs that read
            // it have completed (one commit) and every row warp has taken the tile's metadata
            mbar_init(&sm.empty[s], TC ? 1 + tc_row_warps : kConsumerWarps);
        }
        if constexpr (TC) {
            for (int b = 0; b < kTcSBufs; ++b) {
                mbar_init(&sm.v.bar_s[b], 1);
                mbar_init(&sm.v.bar_p[b], tc_row_warps);
                mbar_init(&sm.v.bar_o[b], 1);
            }
            mbar_init(&sm.v.bar_q, tc_row_warps);
            mbar_init(&sm.v.tmem_done, tc_row_warps);
            for (int b = 0; b < kTcKStages; ++b) mbar_init(&sm.v.empty_k[b], 1);
        }
        mbar_init(&sm.merge_bar[0], TC ? tc_row_warps : NT < kWideTiles ? kConsumerWarps - 1 : kConsumerWarps);   // (rows on M: "partial written" by every warp with rows)
        mbar_init(&sm.merge_bar[1], 1);
        mbar_init(&sm.end_bar, kConsumerWarps);
        mbar_init(&sm.list_bar, kConsumerWarps);
        mbar_init(&sm.land_bar, 1);
        mbar_fence_init();
        sm.issued = 0;
        sm.first_unit = -2;
        sm.pieces_n = 0;
    }
    if (warp == kConsumerWarps && lane == 0) {
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
    }

#ifdef SEER_DECODE_TRACE
    if (tid == 0) {
        unsigned int smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        p.trace[(size_t)blockIdx.x * kTraceSlots + 15] = smid;
    }
#endif
    if (tid == 0) SEER_STAMP(8);
    if constexpr (TC) {
        if (warp == kConsumerWarps + 1) tmem_alloc(&sm.v.tmem_base, kTcCols);
        tc_fence_before_sync();
    }
    __syncthreads();                                 // barriers initialised
    if constexpr (TC) tc_fence_after_sync();
    // The producer warp puts its wait off when the lists' lengths follow from the sequence lengths: it then
    // makes the schedule and finds its first unit while the kernel that writes the lists is still running, and
    // waits just before it reads a list.  (Everything it touches before that was final before that kernel began.)
    bool producer_waited = !(SPARSE && p.sel_from_lens > 0 && warp == kConsumerWarps);
    if (producer_waited) pdl_wait();
    if (tid == 0) SEER_STAMP(9);

    if (warp == kConsumerWarps) {
        // =========================== producer warp ====================================
        // The warp first sums the units' tile counts by itself (the consumer warps do not need the
        // result to start waiting) and derives the schedule.  The prefix sums of the counts, by which
        // the unit that holds a given tile is found, stay in shared memory for up to kSmemUnits units
        // and go through global memory beyond that.
        const int per = (U + 31) / 32;
        const int u_lo = min(U, lane * per), u_hi = min(U, u_lo + per);
        const bool smem_pfx = U <= kSmemUnits;
        int mine = 0, t_min = 0x7fffffff, t_max = 0;
#pragma unroll 1
        for (int u = u_lo; u < u_hi; ++u) {
            const int t = tiles_of<SPARSE, SMALL>(p, u);
            if (t == 0 && cta == 0) write_zero_unit(p, u);       // units without work: zeros, -inf
            if (smem_pfx) sm.upfx[u + 1] = t;                      // (the count for now)
            mine += t;
            t_min = min(t_min, t);
            t_max = max(t_max, t);
        }
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const int T = __shfl_sync(0xffffffffu, incl, 31);
        if (lane == 0) SEER_STAMP(11);
        // With little work (a few tiles per CTA at most) fewer CTAs take part, kMinTiles tiles or more each:
        // a unit is then cut into fewer pieces and its combine is short.  If, moreover, all units have
        // the same number of tiles t, the ranges are made to divide the units evenly (P ranges of t/P
        // tiles per unit, P the largest such divisor of t), so that no range straddles two units --
        // provided that keeps at least 4/5 of the CTAs the plain rule would use.
        int ranges = gridDim.x;
        if (T > 0 && T <= kFewTilesPerCta * (int)gridDim.x && p.min_tiles > 0) {
            ranges = max(1, min((int)gridDim.x, (T + p.min_tiles - 1) / p.min_tiles));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                t_min = min(t_min, __shfl_xor_sync(0xffffffffu, t_min, o));
                t_max = max(t_max, __shfl_xor_sync(0xffffffffu, t_max, o));
            }
            if (t_min == t_max && U <= ranges) {
                const int p_max = max(1, min(ranges / U, t_max / p.min_tiles));
                const int cand = p_max - lane;                   // lane k tries P = p_max - k
                const bool ok = cand >= 1 && t_max % cand == 0;
                const unsigned m = __ballot_sync(0xffffffffu, ok);
                if (m) {
                    const int P = p_max - (__ffs(m) - 1);
                    if (5 * U * P >= 4 * ranges) ranges = U * P;
                }
            }
        }
        Schedule sc;                                     // (its table stays in shared memory)
        build_schedule(sc, sm.sched, T, ranges, p.max_rounds > 0 ? p.pool_div : 0, min(max(p.max_rounds, 1), kMaxRounds), lane);     // (the consumers use it when a piece ends)
        const int R = sc.R, G = sc.G;
        {
            int acc = incl - mine;
            if (smem_pfx) {
                if (lane == 0) sm.upfx[0] = 0;
#pragma unroll 1
                for (int u = u_lo; u < u_hi; ++u) { acc += sm.upfx[u + 1]; sm.upfx[u + 1] = acc; }
            } else if (R > 0) {
                // (every CTA writes the same values; a CTA only relies on its own writes)
#pragma unroll 1
                for (int u = u_lo; u < u_hi; ++u) { p.prefix[u] = acc; acc += tiles_of<SPARSE, SMALL>(p, u); }
                if (lane == 0) p.prefix[U] = T;
            }
            __syncwarp();
        }
        // Unit cu that holds global tile t, with the global index cpu of its first tile and its tile
        // count cut.  false: no unit holds it (the counts changed under us).
        int cu = 0, cpu = 0, cut = 0;
        auto locate = [&](int t, bool first) -> bool {
            int f_u = -1, f_p = 0, f_t = 0;
            if (smem_pfx) {
#pragma unroll 1
                for (int u = u_lo; u < u_hi; ++u) {
                    const int lo = sm.upfx[u], hi = sm.upfx[u + 1];
                    if (lo <= t && t < hi) { f_u = u; f_p = lo; f_t = hi - lo; }
                }
            } else if (first) {
                int acc = incl - mine;
#pragma unroll 1
                for (int u = u_lo; u < u_hi; ++u) {
                    const int n = tiles_of<SPARSE, SMALL>(p, u);
                    if (acc <= t && t < acc + n) { f_u = u; f_p = acc; f_t = n; }
                    acc += n;
                }
            } else {
                // 32-ary search in the prefix sums
                int lo = 0, hi = U;                       // prefix[lo] <= t < prefix[hi]
                while (hi - lo > 1) {
                    const int step = (hi - lo + 31) / 32;
                    const int cand = lo + min((lane + 1) * step, hi - lo);
                    const int pv = cand < hi ? __ldcg(p.prefix + cand) : 0x7fffffff;
                    const unsigned m = __ballot_sync(0xffffffffu, pv > t);
                    const int f = __ffs(m) - 1;             // the last lane always votes yes
                    const int new_hi = __shfl_sync(0xffffffffu, cand, f);
                    const int new_lo = f == 0 ? lo : __shfl_sync(0xffffffffu, cand, f - 1);
                    hi = new_hi;
                    lo = new_lo;
                }
                f_p = __ldcg(p.prefix + lo);
                f_t = __ldcg(p.prefix + lo + 1) - f_p;
                f_u = (t >= f_p && t < f_p + f_t) ? lo : -1;
            }
            const unsigned m = __ballot_sync(0xffffffffu, f_u >= 0);
            if (!m) return false;
            const int src = __ffs(m) - 1;
            cu = __shfl_sync(0xffffffffu, f_u, src);
            cpu = __shfl_sync(0xffffffffu, f_p, src);
            cut = __shfl_sync(0xffffffffu, f_t, src);
            return true;
        };
        int it = 0;
        int iv_begin = 0, iv_end = 0, iv_id = 0;
        bool first = true;               // the static share has not been taken yet
        bool own = R > 0 && cta < G;     // the own range may still have chunks to claim
        bool contiguous = false;         // the next interval continues the previous one
        int fails = 0, steals = 0;
        // What the next interval needs from global memory is asked for before the tiles of the current
        // one are issued, so that the round trip runs under them: the claim on the own range's counter
        // while that range lasts, afterwards the look at all ranges' counters.
        constexpr int kScan = 10;        // counters per lane and round: 320 ranges a round
        int next_own_tiles = 0;          // size of the own range's chunk after the current one
        int ahead = 0;                   // 0: nothing asked for, 1: own claim (pend_old), 2: first round of counters (st)
        int pend_old = 0;
        int st[kScan];
        // (a range's last chunk is left to its owner: by the time a thief's loads came back the owner
        // would have been there)
        const int min_left = min(2, R);
        auto scan_load = [&](int c0) {
#pragma unroll
            for (int k = 0; k < kScan; ++k) {
                const int cc = c0 + 32 * k + lane;
                st[k] = cc < G ? __ldcg(p.steal + cc) : (R << 16);
            }
        };
        auto scan_pick = [&](int c0, int best) -> int {
#pragma unroll
            for (int k = 0; k < kScan; ++k) {
                const int cc = c0 + 32 * k + lane;
                const int left = R - (st[k] & 0xffff) - (st[k] >> 16);
                if (cc < G && cc != cta && left >= min_left) {
                    const int rot = cc - cta + (cc < cta ? G : 0);   // this thief's order of preference
                    best = max(best, (left << 20) | (0xfffff - min(rot, 0xfffff)));
                }
            }
            return best;
        };
        for (;;) {
            {
                int c = 0, j = 0;
                if (first) {
                    // the static share: the head of the own range
                    if (T == 0 || cta >= G) {
                        if (lane == 0) sm.first_unit = -1;
                        break;
                    }
                    c = cta;
                } else if (R == 0) {
                    break;
                } else {
                    bool got = false, done = false;
                    while (!got && !done) {
                        if (own) {
                            // own range, from the front: low half of the counter counts front claims
                            if (ahead != 1 && lane == 0) pend_old = atomicAdd(&p.steal[cta], 1);
                            ahead = 0;
                            const int old = __shfl_sync(0xffffffffu, pend_old, 0);
                            const int taken = (old & 0xffff) + (old >> 16);
                            if (taken + 1 >= R) own = false;     // the last chunk, or none left
                            if (taken >= R) continue;
                            c = cta;
                            j = (old & 0xffff) + 1;
                            contiguous = true;
                            got = true;
                        } else {
                            // Somebody else's range, from the back.  Look at every range's claim counter
                            // and go for the one with the most chunks left (its owner is the furthest
                            // behind); ties are broken differently by every thief.  (All of a lane's
                            // counters are requested before any is looked at: one round trip.)
                            if (fails >= 3 || steals >= kMaxSteals) { done = true; break; }
                            int best = -1;
                            for (int c0 = 0; c0 < G; c0 += 32 * kScan) {
                                if (c0 > 0 || ahead != 2) scan_load(c0);
                                best = scan_pick(c0, best);
                            }
                            ahead = 0;
#pragma unroll
                            for (int off = 16; off > 0; off >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, off));
                            if (best < 0) { done = true; break; }                 // nothing left anywhere
                            c = cta + (0xfffff - (best & 0xfffff));
                            if (c >= G) c -= G;
                            int old = 0;
                            if (lane == 0) old = atomicAdd(&p.steal[c], 1 << 16);
                            old = __shfl_sync(0xffffffffu, old, 0);
                            if ((old & 0xffff) + (old >> 16) >= R) { ++fails; continue; }
                            fails = 0;
                            ++steals;
                            j = R - (old >> 16);
                            contiguous = false;
                            got = true;
                        }
                    }
                    if (!got) break;
                }
                interval_range(sc, sm.sched.off, c, j, &iv_begin, &iv_end);
                iv_id = c * (R + 1) + j;
                if (own && c == cta && j < R) {
                    int nb, ne;
                    interval_range(sc, sm.sched.off, c, j + 1, &nb, &ne);
                    next_own_tiles = ne - nb;
                }
                if (!contiguous) {
                    const bool found = iv_begin < iv_end && locate(iv_begin, first);
                    if (first) {
                        // the consumers request this unit's queries now, ahead of the tile loads that
                        // are about to fill the memory system's queues
                        if (lane == 0) { sm.first_unit = found ? cu : -1; SEER_STAMP(12); }
                        first = false;
                        if (!found) break;
                    } else if (!found) {
                        break;                                // counts changed under us
                    }
                }
            }
            // asks for what the next interval will need (called when the last few tiles of the current
            // interval are about to be issued: earlier, an own claim would take a chunk out of the
            // thieves' reach long before its owner gets to it)
            auto ask_ahead = [&]() {
                if (R == 0) return;
                if (own) {
                    // (only when the chunk to come is small: a big one is worth more within the thieves'
                    // reach than the round trip its claim costs)
                    if (next_own_tiles <= kAheadMaxChunk) {
                        if (lane == 0) pend_old = atomicAdd(&p.steal[cta], 1);
                        ahead = 1;
                    }
                } else if (fails < 3 && steals < kMaxSteals) {
                    scan_load(0);
                    ahead = 2;
                }
            };
            if (!producer_waited && !p.list_flags) {  // the lists are read from here on
                pdl_wait();
                producer_waited = true;
            }
            const bool fresh = !contiguous;          // this interval starts a new piece
            int ce = iv_begin - cpu;                  // offset of the next tile inside unit cu
            const int n_tiles = iv_end - iv_begin;
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
                        cut = tiles_of<SPARSE, SMALL>(p, cu);
                        continue;
                    }
                    int take = min(avail, n_chunk - base);
                    if (lane >= base && lane < base + take) {
                        my_u = cu; my_e = ce + lane - base; my_ut = cut; my_pu = cpu;
                    }
                    base += take;
                    ce += take;
                }
                // per-lane tile descriptor (row/outer: TMA coordinates of the tile, or of each gathered block)
                const int bpt = SMALL ? p.blocks_per_tile : 1;           // (a compile-time 1 for blocks of 64 or 128 tokens)
                int nvalid = 0, head = 0, flags = 0;
                int row[4] = {0, 0, 0, 0}, outer[4] = {0, 0, 0, 0};
                if (my_u >= 0) {
                    const int i = unit_seq(p, my_u);
                    head = my_u - i * p.num_kv_heads;
                    const int L = p.seq_lens[i];
                    if (SPARSE && p.list_flags) {
                        // The gate kernel of the same step marks every unit whose list it has written: the tiles of
                        // the early units are requested while it is still selecting for the late ones.  (That kernel
                        // was launched before this one and all of its CTAs were resident before this one could start,
                        // so it makes progress whatever this warp does; the wait is bounded all the same.)
                        for (int spin = 0; ld_acquire_gpu(p.list_flags + my_u) != p.list_gen; ++spin) {
                            if (spin > (1 << 20)) { raise_status(p.status, DEV_TIMEOUT); break; }
                            __nanosleep(40);
                        }
                    }
                    if (SMALL) {
                        // a tile gathers the next bpt listed blocks of the unit
                        const int n_i = (L + p.block_size - 1) >> p.bs_shift;
                        int cnt_u = p.sel_from_lens > 0 ? min(p.sel_from_lens, n_i) : p.block_cnt ? p.block_cnt[my_u] : p.max_sel;
                        cnt_u = max(0, min(cnt_u, p.max_sel));
#pragma unroll
                        for (int sb = 0; sb < 4; ++sb) {
                            const int e = my_e * bpt + sb;
                            if (sb < bpt && e < cnt_u) {
                                const int blk = p.block_idx[(size_t)my_u * p.max_sel + e];
                                if (blk >= n_i) raise_status(p.status, DEV_BAD_INDEX);
                                if (blk >= 0 && blk < n_i) {
                                    const int tok0 = blk * p.block_size;
                                    int nv = max(0, min(p.block_size + 7, L - tok0));
                                    if (PAGED && nv > 0) {
                                        const int pg = p.page_table[(size_t)i * p.page_table_stride + tok0 / p.page_size];
                                        if (pg < 0 || pg >= p.num_pages) {
                                            raise_status(p.status, DEV_BAD_INDEX);
                                            nv = 0;
                                        }
                                        outer[sb] = pg;
                                        row[sb] = tok0 % p.page_size;
                                    } else {
                                        outer[sb] = i;
                                        row[sb] = tok0;
                                    }
                                    nvalid |= nv << (8 * sb);
                                }
                            }
                        }
                    } else {
                        int tok0 = 0;
                        if (SPARSE) {
                            const int blk = p.block_idx[(size_t)my_u * p.max_sel + (my_e >> p.tpb_shift)];
                            const int n_i = (L + p.block_size - 1) >> p.bs_shift;
                            if (blk >= n_i) raise_status(p.status, DEV_BAD_INDEX);
                            if (blk >= 0 && blk < n_i) {
                                tok0 = (blk << p.bs_shift) + (my_e & (p.tiles_per_block - 1)) * kTileTokens;
                                nvalid = max(0, min(kTileTokens + 7, L - tok0));
                            }
                        } else {
                            tok0 = my_e * kTileTokens;
                            nvalid = max(0, min(kTileTokens + 7, L - tok0));
                        }
                        if (PAGED) {
                            if (nvalid > 0) {
                                const int pg = p.page_table[(size_t)i * p.page_table_stride + tok0 / p.page_size];
                                if (pg < 0 || pg >= p.num_pages) {
                                    raise_status(p.status, DEV_BAD_INDEX);
                                    nvalid = 0;
                                }
                                outer[0] = pg;
                                row[0] = tok0 % p.page_size;
                            }
                        } else {
                            outer[0] = i;
                            row[0] = tok0;
                        }
                    }
                    // bit 0: first tile of a piece; (the piece's end is found by the consumers)
                    flags = (my_e == 0 || (fresh && t + lane == 0)) ? 1 : 0;
                } else if (lane < n_chunk) {
                    // the counts changed under us: keep the pipeline protocol, load nothing
                    my_u = 0; my_ut = 1; flags = 1;
                    raise_status(p.status, DEV_BAD_INDEX);
                }
                for (int s = 0; s < n_chunk; ++s, ++it) {
                    if (n_tiles - (t + s) == min(n_tiles, kAheadTiles)) ask_ahead();
                    const int s_nvalid = __shfl_sync(0xffffffffu, nvalid, s);
                    const int s_head = __shfl_sync(0xffffffffu, head, s);
                    const int s_flags = __shfl_sync(0xffffffffu, flags, s);
                    const int s_u = __shfl_sync(0xffffffffu, my_u, s);
                    const int s_pu = __shfl_sync(0xffffffffu, my_pu, s);
                    const int s_ut = __shfl_sync(0xffffffffu, my_ut, s);
                    int s_row[4], s_outer[4];
#pragma unroll
                    for (int sb = 0; sb < 4; ++sb) {
                        s_row[sb] = (sb == 0 || SMALL) ? __shfl_sync(0xffffffffu, row[sb], s) : 0;
                        s_outer[sb] = (sb == 0 || SMALL) ? __shfl_sync(0xffffffffu, outer[sb], s) : 0;
                    }
                    if (lane == 0) {
                        const int st = it % kS;
#ifdef SEER_DECODE_TRACE
                        if (it == 0) SEER_STAMP(13);
                        if (it == 1) SEER_STAMP(14);
#endif
                        if (!mbar_wait(&sm.empty[st], ((it / kS) & 1) ^ 1, p.status)) return;
                        sm.meta[st] = StageMeta{s_nvalid, s_u, s_flags, s_pu, s_ut, iv_id};
                        __threadfence_block();
                        sm.issued = it + 1;                  // consumers may look ahead at this tile
                        unsigned char* dst = sm.stage[st];
                        if (SMALL && s_nvalid > 0) {
                            // one box of b rows per gathered block, at its place in the 64-row tile
                            const int sub_bytes = p.block_size * 128;        // one half (64 channels) of one block
                            int n_sub = 0;
#pragma unroll
                            for (int sb = 0; sb < 4; ++sb) n_sub += ((s_nvalid >> (8 * sb)) & 0xff) ? 1 : 0;
                            mbar_arrive_expect_tx(&sm.full[st], (uint32_t)(n_sub * 4 * sub_bytes));
#pragma unroll
                            for (int sb = 0; sb < 4; ++sb) {
                                if ((s_nvalid >> (8 * sb)) & 0xff) {
                                    unsigned char* d2 = dst + sb * sub_bytes;
                                    tma_load_4d(d2, &map_k, &sm.full[st], 0, s_row[sb], s_head, s_outer[sb]);
                                    tma_load_4d(d2 + kHalfTileBytes, &map_k, &sm.full[st], 64, s_row[sb], s_head, s_outer[sb]);
                                    tma_load_4d(d2 + kTileBytes, &map_v, &sm.full[st], 0, s_row[sb], s_head, s_outer[sb]);
                                    tma_load_4d(d2 + kTileBytes + kHalfTileBytes, &map_v, &sm.full[st], 64, s_row[sb],
                                                s_head, s_outer[sb]);
                                }
                            }
                        } else if (TC) {
                            // K and V go to rings of their own: the K buffer has to be free as well
                            if constexpr (TC) {
                                const int sk = it % kTcKStages;
                                if (!mbar_wait(&sm.v.empty_k[sk], ((it / kTcKStages) & 1) ^ 1, p.status)) return;
                                if (s_nvalid > 0) {
                                    unsigned char* dk = sm.stage[0] + (size_t)(kTcStages + sk) * kTileBytes;
                                    unsigned char* dv = sm.stage[0] + (size_t)st * kTileBytes;
                                    mbar_arrive_expect_tx(&sm.full[st], kStageBytes);
                                    tma_load_4d(dk, &map_k, &sm.full[st], 0, s_row[0], s_head, s_outer[0]);
                                    tma_load_4d(dk + kHalfTileBytes, &map_k, &sm.full[st], 64, s_row[0], s_head, s_outer[0]);
                                    tma_load_4d(dv, &map_v, &sm.full[st], 0, s_row[0], s_head, s_outer[0]);
                                    tma_load_4d(dv + kHalfTileBytes, &map_v, &sm.full[st], 64, s_row[0], s_head, s_outer[0]);
                                } else {
                                    mbar_arrive(&sm.full[st]);
                                }
                            }
                        } else if (s_nvalid > 0) {
                            mbar_arrive_expect_tx(&sm.full[st], kStageBytes);
                            tma_load_4d(dst, &map_k, &sm.full[st], 0, s_row[0], s_head, s_outer[0]);
                            tma_load_4d(dst + kHalfTileBytes, &map_k, &sm.full[st], 64, s_row[0], s_head, s_outer[0]);
                            tma_load_4d(dst + kTileBytes, &map_v, &sm.full[st], 0, s_row[0], s_head, s_outer[0]);
                            tma_load_4d(dst + kTileBytes + kHalfTileBytes, &map_v, &sm.full[st], 64, s_row[0],
                                        s_head, s_outer[0]);
                        } else {
                            mbar_arrive(&sm.full[st]);
                        }
                    }
                }
            }
        }
        if (!producer_waited) pdl_wait();            // (a CTA without tiles: the counters below belong to this launch only after the wait)
        if (lane == 0) {
            // end-of-stream marker for the consumers
            const int st = it % kS;
            if (!mbar_wait(&sm.empty[st], ((it / kS) & 1) ^ 1, p.status)) return;
            sm.meta[st] = StageMeta{-1, -1, 1, 0, 0, 0};
            __threadfence_block();
            sm.issued = it + 1;
            mbar_arrive(&sm.full[st]);
            // the last CTA to stop claiming work re-arms the counters for the next launch
            __threadfence();
            if (atomicAdd(&p.sched[1], 1) == (int)gridDim.x - 1) {
                for (int c = 0; c < (int)gridDim.x; ++c) p.steal[c] = 0;
                p.sched[0] = 0;
                p.sched[1] = 0;
            }
        }
        return;
    }

    if constexpr (TC) {
    if (warp == kConsumerWarps + 1) {
        // =========================== MMA warp (tensor-memory variant) ====================
        // Lane 0 issues, per tile, S = Q . K^T (8 MMAs of K = 16 over the 128 channels; Q from tensor memory,
        // where the row warps put the unit's queries when a piece begins, the K tile K-major in shared
        // memory) and, once the row warps have written the tile's probabilities, O (+)= P . V (4 MMAs over
        // the 64 tokens; P from tensor memory, the V tile MN-major).  The tensor cores work on S(t + 1)
        // while the row warps are busy with S(t).  The whole warp clears the rows of a ragged last tile of V.
        const uint32_t tbase = sm.v.tmem_base;
        const uint32_t t_o = tbase + kTcOCol;
        constexpr uint32_t idesc_qk = tc_idesc_bf16(kTcRows, kTileTokens, false);
        constexpr uint32_t idesc_pv = tc_idesc_bf16(kTcRows, kHeadDim, true);
        const uint32_t t_q = tbase + kTcQCol;
        int piece_no = 0;                          // pieces begun so far (phase of bar_q)
        bool dead = false;                         // a wait ran out: stop issuing, free the tensor memory, leave
        int ct = 0, piece_ct = 0;                  // computed tiles so far (of the CTA, of the piece)
#ifdef SEER_DECODE_TRACE
        unsigned long long mm_tr[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        const long long mm_t0 = clock64();
#endif
        // Two kinds of work, taken as they become possible: the scores of the next tile once it has landed
        // (at most three tiles may be between their scores and their product: S has three buffers), and the
        // product of the oldest such tile once its probabilities are written.  A stage is released by the
        // commit behind its product, so it is held no longer than the row warps need for its tile.
        int pend_n = 0;                            // tiles whose product is still to be issued (0..kTcSBufs)
        int pend_stage[kTcSBufs] = {};
        bool pend_acc[kTcSBufs] = {};              // indexed by the tile's S buffer (ct % kTcSBufs)
        int it = 0;                                // next tile of the stream
        bool ended = false;
        uint32_t idle = 0;
        while (!dead && (!ended || pend_n > 0)) {
            bool did = false;
            if (pend_n > 0) {
                const int c = ct - pend_n, b = c % kTcSBufs;
                if (__shfl_sync(0xffffffffu, lane == 0 ? (int)mbar_test_wait(&sm.v.bar_p[b], (c / kTcSBufs) & 1) : 0, 0)) {
                    __syncwarp();
                    if (lane == 0) {
                        tc_fence_after_sync();
                        const uint32_t v_addr = smem_u32(sm.stage[0]) + pend_stage[b] * kTileBytes;
#pragma unroll
                        for (int ks = 0; ks < kTileTokens / 16; ++ks)
                            tc_mma_ts(t_o, tbase + 64 * b + 8 * ks, tc_smem_desc(v_addr + ks * 2048, kHalfTileBytes, 1024), idesc_pv,
                                      pend_acc[b] || ks > 0);
                        tc_commit(&sm.empty[pend_stage[b]]);   // the stage's K and V have been read
                        tc_commit(&sm.v.bar_o[b]);
                    }
                    __syncwarp();
                    --pend_n;
                    did = true;
                }
            }
            if (!ended && pend_n < kTcSBufs) {
                const int st = it % kS;
                if (__shfl_sync(0xffffffffu, lane == 0 ? (int)mbar_test_wait(&sm.full[st], (it / kS) & 1) : 0, 0)) {
                    // (every lane reads the metadata after lane 0 has seen the barrier's phase complete)
                    mbar_try_wait(&sm.full[st], (it / kS) & 1);
                    __syncwarp();
                    const StageMeta mt = sm.meta[st];
                    // the first tile of a piece has to find the piece's queries in tensor memory
                    const bool q_ready = mt.nvalid < 0 || !(mt.flags & 1) ||
                        __shfl_sync(0xffffffffu, lane == 0 ? (int)mbar_test_wait(&sm.v.bar_q, piece_no & 1) : 0, 0);
                    if (q_ready) {
                    did = true;
                    if (mt.nvalid < 0) {
                        ended = true;
                    } else {
                        if (mt.flags & 1) { piece_ct = 0; ++piece_no; }
                        const int nv = mt.nvalid;
                        if (nv > 0) {
                            if (nv < kTileTokens) {
                                // ragged tail: rows past the sequence end may hold anything; cleared in V so that a
                                // zero probability times garbage cannot produce NaN
                                unsigned char* vt = sm.stage[0] + (size_t)st * kTileBytes;
                                for (int x = lane; x < (kTileTokens - nv) * 16; x += 32) {
                                    const int r = nv + (x >> 4), part = x & 15;
                                    *reinterpret_cast<uint4*>(vt + (part >> 3) * kHalfTileBytes + r * 128 + ((part & 7) << 4)) =
                                        make_uint4(0u, 0u, 0u, 0u);
                                }
                                fence_proxy_async_smem();
                                __syncwarp();
                            }
                            const int b = ct % kTcSBufs;
                            if (lane == 0) {
                                tc_fence_after_sync();
                                const uint32_t k_addr = smem_u32(sm.stage[0]) + (kTcStages + it % kTcKStages) * kTileBytes;
#pragma unroll
                                for (int ks = 0; ks < kHeadDim / 16; ++ks)
                                    tc_mma_ts(tbase + 64 * b, t_q + 8 * ks,
                                              tc_smem_desc(k_addr + (ks >> 2) * kHalfTileBytes + (ks & 3) * 32, 16, 1024), idesc_qk, ks > 0);
                                tc_commit(&sm.v.bar_s[b]);
                                tc_commit(&sm.v.empty_k[it % kTcKStages]);   // the K buffer has been read
                            }
                            __syncwarp();
                            pend_stage[b] = st;
                            pend_acc[b] = piece_ct > 0;
                            ++pend_n;
                            ++ct;
                            ++piece_ct;
                        } else {
                            if (lane == 0) {                               // nothing was loaded: the buffers go straight back
                                mbar_arrive(&sm.empty[st]);
                                mbar_arrive(&sm.v.empty_k[it % kTcKStages]);
                            }
                        }
                        ++it;
                    }
                    }
                }
            }
            if (did) {
                idle = 0;
            } else if (++idle > 64) {
                if (idle > (1u << 23)) {               // seconds: whatever this warp waits for will not come
                    raise_status(p.status, DEV_TIMEOUT);
                    dead = true;
                }
                __nanosleep(32);
            }
        }
#ifdef SEER_DECODE_TRACE
        mm_tr[3] = (unsigned long long)(clock64() - mm_t0);
        if (lane == 0) for (int k = 0; k < 8; ++k) p.trace[(size_t)blockIdx.x * kTraceSlots + 64 + k] = mm_tr[k];
#endif
        // the tensor memory goes back once the row warps are done with it (or a wait has run out)
        mbar_wait(&sm.v.tmem_done, 0, p.status);
        __syncwarp();
        tmem_dealloc(tbase, kTcCols);
        return;
    }
    }

    // =============================== consumer warps =====================================
    const int w = warp;
    const int qd = lane & 3;            // column pair: rows 2*qd, 2*qd+1 of every N-tile
    const int rw = lane >> 2;           // row within an 8-row slab
    unsigned long long tk_before = 0ull; // warp 0, lane k: what the unit's counter held before the k-th held piece was added
    unsigned int tk_bit = 0u;            // ... and that piece's bit
    int piece_tiles = 0, piece_iv = 0;  // tiles in the current piece, interval it started in
    if constexpr (TC) {
    // ---------------- the unit's rows on M, on the fifth-generation tensor cores ----------------
    // Thread t of the four row warps is row t of the unit and lane t of tensor memory; warps whose 32 rows
    // are all padding have nothing to do until the stream is over.  Per tile a row thread reads its 64 scores
    // (S, fp32), masks, exponentiates against the row's reference maximum, adds up, and writes the 64
    // probabilities back over S as bf16 pairs (P) for the MMA warp's second product.  The reference maximum
    // only moves when the true one has grown by more than 2^8 since (probabilities stay below 2^8, exact in
    // bf16's range); O, which accumulates in tensor memory, is rescaled on those occasions only.
    //     S (128 x 64 tok) = Q (128 x 128) . K^T      tcgen05.mma, Q from tensor memory, K K-major in shared memory
    //     O (128 x 128)   += P (128 x 64) . V          P from tensor memory, V MN-major in shared memory
    constexpr float kSlack = 8.f;
#ifdef SEER_DECODE_TRACE
    unsigned long long tc_tr[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#define TC_T(v) const long long v = clock64()
#define TC_ACC(k, a, b) tc_tr[k] += (unsigned long long)((b) - (a))
#else
#define TC_T(v)
#define TC_ACC(k, a, b)
#endif
    const int row = tid;
    const bool real = row < p.rows;
    // newest cached tokens the row may not see (its query token's distance from the last one)
    const int back = real ? p.q_len - 1 - (p.t_base + ((row * p.group_magic) >> 16)) : 0;
    int pubs = 0;                       // partials written so far (phase of merge_bar[0])
    if (32 * w < p.rows) {
        const uint32_t tbase = sm.v.tmem_base + ((uint32_t)(32 * w) << 16);
        const uint32_t t_o = tbase + kTcOCol;
        float m_ref = -INFINITY, l_run = 0.f;
        int ct = 0, piece_ct = 0;       // computed tiles so far (of the CTA, of the piece)
        // A piece's queries go to tensor memory, this thread's row as 64 columns of bf16 pairs (zeros for a padding
        // row): requested from global memory early, stored once every score of the piece before has been computed
        // (this thread has then read the last of them); the MMA warp issues none of the new piece's before all
        // row warps have arrived.
        auto load_q = [&](int unit, uint4 (&qv)[16]) {
            const uint4* qsrc = reinterpret_cast<const uint4*>(p.q + unit_row(p, unit, real ? row : 0) * kHeadDim);
#pragma unroll
            for (int x = 0; x < 16; ++x) qv[x] = real ? __ldg(qsrc + x) : make_uint4(0u, 0u, 0u, 0u);
        };
        auto store_q = [&](const uint4 (&qv)[16]) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t qr[32];
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    qr[4 * x] = qv[8 * h + x].x; qr[4 * x + 1] = qv[8 * h + x].y;
                    qr[4 * x + 2] = qv[8 * h + x].z; qr[4 * x + 3] = qv[8 * h + x].w;
                }
                tmem_st32(tbase + kTcQCol + 32 * h, qr);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.v.bar_q);
        };
        if (!mbar_wait(&sm.full[0], 0, p.status)) return;
        if (tid == 0) SEER_STAMP(10);
        StageMeta mt = sm.meta[0];
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.empty[0]);              // metadata taken
        for (int it = 0; mt.nvalid >= 0; ++it) {
            if (mt.flags & 1) {
                m_ref = -INFINITY;
                l_run = 0.f;
                piece_tiles = 0;
                piece_iv = mt.interval;
                piece_ct = 0;
                // (the first piece's queries; those of a later piece are put in place when the piece before it ends)
                if (it == 0) {
                    uint4 qv[16];
                    load_q(mt.unit, qv);
                    store_q(qv);
                }
            }
            ++piece_tiles;
            const int nv = mt.nvalid;                          // cached tokens from the tile's first row on (capped at 64 + 7)
            if (nv > 0) {
                const int b = ct % kTcSBufs;
                TC_T(t_a);
                if (!mbar_wait(&sm.v.bar_s[b], (ct / kTcSBufs) & 1, p.status)) return;
                __syncwarp();
                tc_fence_after_sync();
                TC_T(t_b);
                TC_ACC(0, t_a, t_b);
                uint32_t sr[2][32];
                tmem_ld32(tbase + 64 * b, sr[0]);
                tmem_ld32(tbase + 64 * b + 32, sr[1]);
                tmem_wait_ld();
                TC_T(t_c);
                TC_ACC(1, t_b, t_c);
                // tokens the row may see: the first `lim` of the tile; hidden ones get a score of -inf.  (Only the
                // newest tiles of a sequence have any, so the test is skipped when the whole warp sees all 64.)
                const int lim = nv - back;
                if (!__all_sync(0xffffffffu, lim >= kTileTokens)) {
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (32 * h + c >= lim) sr[h][c] = 0xff800000u;
                }
                float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};       // (four short chains instead of one long)
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int c = 0; c < 32; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], __uint_as_float(sr[h][c]));
                // (the scale is positive: the largest raw score is the largest scaled one)
                const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
                const float m_new = fmaxf(m_ref, mx);
                const bool grow = m_new > m_ref + kSlack;      // (also: the row's first visible token)
                if (__any_sync(0xffffffffu, grow)) {
#ifdef SEER_DECODE_TRACE
                    tc_tr[4] += 1;
#endif
                    float alpha = 1.f;
                    if (grow) {
                        alpha = m_ref == -INFINITY ? 0.f : fast_exp2(m_ref - m_new);
                        m_ref = m_new;
                        l_run *= alpha;
                    }
                    if (piece_ct > 0) {
                        // O holds the earlier tiles' products: all of them are in once the last one is
                        const int c = ct - 1;
                        if (!mbar_wait(&sm.v.bar_o[c % kTcSBufs], (c / kTcSBufs) & 1, p.status)) return;
                        __syncwarp();
                        tc_fence_after_sync();
#pragma unroll 1
                        for (int q4 = 0; q4 < 4; ++q4) {
                            uint32_t orow[32];
                            tmem_ld32(t_o + 32 * q4, orow);
                            tmem_wait_ld();
#pragma unroll
                            for (int c2 = 0; c2 < 32; ++c2) orow[c2] = __float_as_uint(__uint_as_float(orow[c2]) * alpha);
                            tmem_st32(t_o + 32 * q4, orow);
                        }
                    }
                }
                // a row that has seen nothing so far keeps max = -inf; exponents are then taken against 0
                const float mb = m_ref == -INFINITY ? 0.f : m_ref;
                float sum4[4] = {0.f, 0.f, 0.f, 0.f};
                uint32_t pk[32];
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(sr[h][c]), p.scale_log2, -mb));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(sr[h][c + 1]), p.scale_log2, -mb));
                        sum4[(c >> 1) & 3] += p0 + p1;
                        pk[(32 * h + c) >> 1] = pack_bf16x2(p0, p1);
                    }
                const float sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
                l_run += sum;
                tmem_st32(tbase + 64 * b, pk);                 // P over the first half of S's columns
                tmem_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.v.bar_p[b]);
                TC_T(t_d);
                TC_ACC(2, t_c, t_d);
                ++ct;
                ++piece_ct;
            }
            // the next tile's metadata tells whether the piece goes on
            const int nst = (it + 1) % kS;
            TC_T(t_e);
            if (!mbar_wait(&sm.full[nst], ((it + 1) / kS) & 1, p.status)) return;
            const StageMeta nx = sm.meta[nst];
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[nst]);        // metadata taken
            TC_T(t_f);
            TC_ACC(3, t_e, t_f);
            if (nx.flags & 1) {
                // ---------------- the current piece ends here: every row thread stores its row -----------------
                const int u = mt.unit;
                const bool partial = piece_tiles < mt.unit_tiles;
                // the next piece's queries travel while this piece's last product completes; once they are in
                // tensor memory the MMA warp computes the next piece's first scores under the read-out below
                const bool more = nx.nvalid >= 0;
                uint4 qv[16];
                if (more) load_q(nx.unit, qv);
                if (piece_ct > 0) {
                    const int c = ct - 1;
                    if (!mbar_wait(&sm.v.bar_o[c % kTcSBufs], (c / kTcSBufs) & 1, p.status)) return;
                    __syncwarp();
                    tc_fence_after_sync();
                }
                if (more) store_q(qv);
                const size_t slot = (size_t)piece_iv + u;
                float* po = p.part_o + slot * (8 * NT * kHeadDim) + row * kHeadDim;
                float* pm = p.part_ml + slot * (kMlStride * NT);
                const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
                const size_t orow_g = unit_row(p, u, real ? row : 0);
#pragma unroll 1
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t orow[32];
                    if (piece_ct > 0) {
                        tmem_ld32(t_o + 32 * q4, orow);
                        tmem_wait_ld();
                    } else {
#pragma unroll
                        for (int c2 = 0; c2 < 32; ++c2) orow[c2] = 0u;
                    }
                    if (real) {
                        if (partial) {
#pragma unroll
                            for (int c2 = 0; c2 < 32; c2 += 4)
                                *reinterpret_cast<uint4*>(po + 32 * q4 + c2) = make_uint4(orow[c2], orow[c2 + 1], orow[c2 + 2], orow[c2 + 3]);
                        } else {
                            uint4* ob = reinterpret_cast<uint4*>(p.out + orow_g * kHeadDim + 32 * q4);
#pragma unroll
                            for (int c2 = 0; c2 < 32; c2 += 8) {
                                ob[c2 >> 3] = make_uint4(
                                    pack_bf16x2(__uint_as_float(orow[c2]) * inv, __uint_as_float(orow[c2 + 1]) * inv),
                                    pack_bf16x2(__uint_as_float(orow[c2 + 2]) * inv, __uint_as_float(orow[c2 + 3]) * inv),
                                    pack_bf16x2(__uint_as_float(orow[c2 + 4]) * inv, __uint_as_float(orow[c2 + 5]) * inv),
                                    pack_bf16x2(__uint_as_float(orow[c2 + 6]) * inv, __uint_as_float(orow[c2 + 7]) * inv));
                            }
                        }
                    }
                }
                if (partial) {
                    if (real) { pm[row] = m_ref; pm[8 * NT + row] = l_run; }
                    if (tid == 0) pm[16 * NT] = __uint_as_float(p.generation);
                    // every row warp makes its rows of the partial visible; then warp 0 counts the piece on the unit's
                    // ticket (lane k for the k-th piece held, answer kept in a register)
                    __threadfence();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.merge_bar[0]);
                    if (w == 0) {
                        if (!mbar_wait(&sm.merge_bar[0], pubs & 1, p.status)) return;
                        const int n_held = sm.pieces_n;
                        if (n_held < kMaxPieces) {
                            if (lane == n_held) {
                                const int iv_first = interval_of(sm.sched, mt.unit_first);
                                const int iv_last = interval_of(sm.sched, mt.unit_first + mt.unit_tiles - 1);
                                const int n_slots = iv_last - iv_first + 1;
                                const unsigned int bit = n_slots <= 32 ? 1u << (piece_iv - iv_first) : 0u;
                                sm.pieces[n_held] = Piece{u, piece_tiles, iv_first + u, n_slots, mt.unit_tiles};
                                tk_bit = bit;
                                tk_before = atomicAdd(&p.tickets[u], ((unsigned long long)piece_tiles << 32) | bit);
                            }
                            __syncwarp();
                            if (lane == 0) sm.pieces_n = n_held + 1;
                        } else {
                            raise_status(p.status, DEV_TIMEOUT);   // (cannot happen with the schedule's bound on pieces per CTA)
                        }
                    }
                    ++pubs;
                } else if (p.lse && real) {
                    p.lse[orow_g] = l_run > 0.f ? (m_ref + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
                }
            }
            mt = nx;
        }
#ifdef SEER_DECODE_TRACE
        if (lane == 0) for (int k = 0; k < 8; ++k) p.trace[(size_t)blockIdx.x * kTraceSlots + 32 + 8 * w + k] = tc_tr[k];
#endif
        // the last access to tensor memory is behind this warp: the MMA warp may give the columns back
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.v.tmem_done);
    }
    } else if constexpr (NT < kWideTiles) {
    // ---------------- tokens on the MMA's M side, the unit's (up to 16) rows on N ----------------
    uint32_t bq[NT][8][2];              // Q^T B-fragments: NT N-tiles x 8 k-steps over d
    uint32_t bq_pre[8][2];              // NT == 1: the same for the unit expected next (prefetched)
    float o[NT][8][4];                  // O^T accumulators: 8 m-tiles over d per N-tile
    float m_run[NT][2], l_run[NT][2];
    int seg = 0;                        // merge rounds finished so far (NT per piece)
    // Query token of this thread's two columns in every N-tile, as the number of newest cached
    // tokens it may not see (q_len - 1 - token): column c of N-tile nt is row 8*nt + c of the unit,
    // i.e. token t_base + row / group.  Rows past p.rows are padding (their result is never stored).
    int back[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            const int r = 8 * nt + 2 * qd + c;
            back[nt][c] = r < p.rows ? p.q_len - 1 - (p.t_base + ((r * p.group_magic) >> 16)) : 0;
        }
    // B fragment of N-tile nt: this thread supplies row 8*nt + rw of the unit's queries
    auto load_q = [&](uint32_t (&dst)[8][2], int unit, int nt) {
        const int r = 8 * nt + rw;
        const bool real = r < p.rows;
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(p.q + unit_row(p, unit, real ? r : 0) * kHeadDim);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            dst[ks][0] = real ? __ldg(qrow + (16 * ks + 2 * qd) / 2) : 0u;
            dst[ks][1] = real ? __ldg(qrow + (16 * ks + 8 + 2 * qd) / 2) : 0u;
        }
    };
    int pre_unit = -1;
    if (NT == 1) {
        // the first tile's unit is known as soon as the producer has found where its share starts,
        // well before the first tile is even requested: ask for that unit's queries at once
        for (int spin = 0; spin < (1 << 22) && sm.first_unit == -2; ++spin) __nanosleep(20);
        const int u0 = sm.first_unit;
        if (u0 >= 0) { load_q(bq_pre, u0, 0); pre_unit = u0; }
    }

    // lane-constant parts of the ldmatrix addresses (swizzle: 16-B chunk ^= row & 7)
    const int k_row = 16 * w + ((lane >> 3) & 1) * 8 + (lane & 7);
    const int k_csel = lane >> 4;                    // which of the two 16-B chunks of a k-step
    const int v_row = 16 * w + ((lane >> 4) & 1) * 8 + (lane & 7);
    const int v_csel = (lane >> 3) & 1;
    const int sw = lane & 7;

    // blocks of 16 or 32 tokens: which of a tile's gathered blocks this warp's rows belong to, and where in it
    constexpr bool small_blocks = SMALL;
    const int sub_w = p.block_size == 16 ? w : (w >> 1), off_w = p.block_size == 16 ? 0 : (w & 1) * 16;
    // the first tile's metadata
    if (!mbar_wait(&sm.full[0], 0, p.status)) return;
    if (tid == 0) SEER_STAMP(10);
    StageMeta mt = sm.meta[0];
    for (int it = 0; mt.nvalid >= 0; ++it) {
        const int st = it % kS;
#ifdef SEER_DECODE_TRACE
        if (tid == 0 && it < kTraceSlots - 16) SEER_STAMP(16 + it);
        if (tid == 0) p.trace[(size_t)blockIdx.x * kTraceSlots + 3] = it + 1;     // tiles consumed so far
#endif
        if (NT == 1) {
            // look ahead: request the queries of the next unit as soon as the producer has issued a
            // tile of it (its metadata is stable from then until we release that stage)
            const int iss = sm.issued;
            __threadfence_block();
#pragma unroll
            for (int look = 1; look < kS; ++look) {
                if (it + look < iss) {
                    const int u2 = *reinterpret_cast<volatile int*>(&sm.meta[(it + look) % kS].unit);
                    if (u2 >= 0 && u2 != mt.unit && u2 != pre_unit) {
                        load_q(bq_pre, u2, 0);
                        pre_unit = u2;
                        break;
                    }
                }
            }
        }
        if (mt.flags & 1) {
            // first tile of a piece: fresh state, the unit's queries
            if (NT == 1 && mt.unit == pre_unit) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) { bq[0][ks][0] = bq_pre[ks][0]; bq[0][ks][1] = bq_pre[ks][1]; }
            } else {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) load_q(bq[nt], mt.unit, nt);
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                for (int a = 0; a < 8; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) o[nt][a][b] = 0.f;
                m_run[nt][0] = m_run[nt][1] = -INFINITY;
                l_run[nt][0] = l_run[nt][1] = 0.f;
            }
            piece_tiles = 0;
            piece_iv = mt.interval;
        }
        ++piece_tiles;
        // mt.nvalid counts the cached tokens from the tile's first row on (up to 7 beyond the tile, so
        // that earlier query tokens can be cut off); nvw is the same count taken from this warp's first
        // row (with blocks of 16 or 32 tokens: from the count of the gathered block the warp's 16 rows
        // belong to)
        const int nvw = small_blocks ? ((mt.nvalid >> (8 * sub_w)) & 0xff) - off_w : mt.nvalid - 16 * w;
        if (nvw > 0) {
            const uint32_t kbase = smem_u32(sm.stage[st]);
            const uint32_t vbase = kbase + kTileBytes;
            if (nvw < 16) {
                // ragged tail: rows past the sequence end may hold anything; clear this warp's
                // V rows so that 0-probability times garbage cannot produce NaN
                unsigned char* vt = sm.stage[st] + kTileBytes;
                for (int x = lane; x < 16 * 32; x += 32) {
                    int r = 16 * w + (x >> 5), part = x & 31;      // 32 x 8-byte pieces per row
                    if ((x >> 5) >= nvw) {
                        int half = part >> 4, off = (part & 15) * 8;
                        *reinterpret_cast<uint2*>(vt + half * kHalfTileBytes + r * 128 + off) =
                            make_uint2(0u, 0u);
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
            }
            // ---- S^T = K . Q^T (two independent accumulator chains per N-tile) ----
            float sa[NT][4], sb[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int x = 0; x < 4; ++x) sa[nt][x] = sb[nt][x] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                uint32_t a[4];
                const int c8 = ((2 * ks) & 7) + k_csel;
                ldmatrix_x4(a, kbase + (ks >> 2) * kHalfTileBytes + k_row * 128 + ((c8 ^ sw) << 4));
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    if (ks & 1) mma_bf16_16816(sb[nt], a, bq[nt][ks][0], bq[nt][ks][1]);
                    else        mma_bf16_16816(sa[nt], a, bq[nt][ks][0], bq[nt][ks][1]);
                }
            }
            const int r0 = rw;                         // row within the warp's 16
            uint32_t pb[NT][2];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                float s[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) s[x] = (sa[nt][x] + sb[nt][x]) * p.scale_log2;
                // a row's token sees the first nvw - back cached tokens counted from this warp's first row
                const int lim0 = nvw - back[nt][0], lim1 = nvw - back[nt][1];
                if (r0 >= lim0) s[0] = -INFINITY;
                if (r0 >= lim1) s[1] = -INFINITY;
                if (r0 + 8 >= lim0) s[2] = -INFINITY;
                if (r0 + 8 >= lim1) s[3] = -INFINITY;
                // ---- online softmax over this warp's 16 tokens, per row (column of S^T) ----
                float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) {
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
                }
                const float mn0 = fmaxf(m_run[nt][0], mx0), mn1 = fmaxf(m_run[nt][1], mx1);
                // a row that has seen nothing so far keeps max = -inf; exponents are then taken against 0
                const float mb0 = mn0 == -INFINITY ? 0.f : mn0, mb1 = mn1 == -INFINITY ? 0.f : mn1;
                const float al0 = fast_exp2(m_run[nt][0] - mb0), al1 = fast_exp2(m_run[nt][1] - mb1);
                // the running maxima rarely move after a piece's first tiles: then nothing is rescaled
                const bool same_max = __all_sync(0xffffffffu, m_run[nt][0] == mn0 && m_run[nt][1] == mn1);
                m_run[nt][0] = mn0; m_run[nt][1] = mn1;
                const float p0 = fast_exp2(s[0] - mb0), p1 = fast_exp2(s[1] - mb1);
                const float p2 = fast_exp2(s[2] - mb0), p3 = fast_exp2(s[3] - mb1);
                l_run[nt][0] = l_run[nt][0] * al0 + (p0 + p2);
                l_run[nt][1] = l_run[nt][1] * al1 + (p1 + p3);
                if (!same_max) {
#pragma unroll
                    for (int a = 0; a < 8; ++a) {
                        o[nt][a][0] *= al0; o[nt][a][1] *= al1; o[nt][a][2] *= al0; o[nt][a][3] *= al1;
                    }
                }
                pb[nt][0] = movmatrix_trans(pack_bf16x2(p0, p1));   // tokens 0-7 of the slice
                pb[nt][1] = movmatrix_trans(pack_bf16x2(p2, p3));   // tokens 8-15
            }
            // ---- O^T += V^T . P^T ----
#pragma unroll
            for (int a = 0; a < 8; ++a) {
                uint32_t f[4];
                const int c8 = ((2 * a) & 7) + v_csel;
                ldmatrix_x4_trans(f, vbase + (a >> 2) * kHalfTileBytes + v_row * 128 + ((c8 ^ sw) << 4));
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) mma_bf16_16816(o[nt][a], f, pb[nt][0], pb[nt][1]);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.empty[st]);

        // the next tile's metadata tells whether the piece goes on
        const int nst = (it + 1) % kS;
        if (!mbar_wait(&sm.full[nst], ((it + 1) / kS) & 1, p.status)) return;
        const StageMeta nx = sm.meta[nst];
        if (nx.flags & 1) {
            // ---------------- the current piece ends here ------------------------------------
            // One merge round per N-tile through the same scratch: warps 1..3 hand (o, max, sum) of the
            // N-tile to warp 0, which folds them into its own.
            float m_all[NT][2], l_all[NT][2];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                float l0 = l_run[nt][0], l1 = l_run[nt][1];
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) {
                    l0 += __shfl_xor_sync(0xffffffffu, l0, off);
                    l1 += __shfl_xor_sync(0xffffffffu, l1, off);
                }
                if (w > 0) {
                    if (seg > 0 && !mbar_wait(&sm.merge_bar[1], (seg - 1) & 1, p.status)) return;   // scratch free?
#pragma unroll
                    for (int a = 0; a < 8; ++a) {
                        const int d0 = 16 * a + rw;
                        sm.v.merge_o[w - 1][2 * qd][d0] = o[nt][a][0];
                        sm.v.merge_o[w - 1][2 * qd + 1][d0] = o[nt][a][1];
                        sm.v.merge_o[w - 1][2 * qd][d0 + 8] = o[nt][a][2];
                        sm.v.merge_o[w - 1][2 * qd + 1][d0 + 8] = o[nt][a][3];
                    }
                    if (rw == 0) {
                        sm.v.merge_ml[w - 1][0][2 * qd] = m_run[nt][0];
                        sm.v.merge_ml[w - 1][0][2 * qd + 1] = m_run[nt][1];
                        sm.v.merge_ml[w - 1][1][2 * qd] = l0;
                        sm.v.merge_ml[w - 1][1][2 * qd + 1] = l1;
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.merge_bar[0]);
                } else {
                    if (!mbar_wait(&sm.merge_bar[0], seg & 1, p.status)) return;
                    float mw[kConsumerWarps - 1][2], lw[kConsumerWarps - 1][2];
                    m_all[nt][0] = m_run[nt][0]; m_all[nt][1] = m_run[nt][1];
#pragma unroll
                    for (int ww = 0; ww < kConsumerWarps - 1; ++ww) {
                        mw[ww][0] = sm.v.merge_ml[ww][0][2 * qd]; mw[ww][1] = sm.v.merge_ml[ww][0][2 * qd + 1];
                        lw[ww][0] = sm.v.merge_ml[ww][1][2 * qd]; lw[ww][1] = sm.v.merge_ml[ww][1][2 * qd + 1];
                        m_all[nt][0] = fmaxf(m_all[nt][0], mw[ww][0]); m_all[nt][1] = fmaxf(m_all[nt][1], mw[ww][1]);
                    }
                    const float f0 = (m_run[nt][0] == -INFINITY) ? 0.f : fast_exp2(m_run[nt][0] - m_all[nt][0]);
                    const float f1 = (m_run[nt][1] == -INFINITY) ? 0.f : fast_exp2(m_run[nt][1] - m_all[nt][1]);
                    l_all[nt][0] = l0 * f0; l_all[nt][1] = l1 * f1;
#pragma unroll
                    for (int a = 0; a < 8; ++a) {
                        o[nt][a][0] *= f0; o[nt][a][1] *= f1; o[nt][a][2] *= f0; o[nt][a][3] *= f1;
                    }
#pragma unroll
                    for (int ww = 0; ww < kConsumerWarps - 1; ++ww) {
                        const float g0 = (mw[ww][0] == -INFINITY) ? 0.f : fast_exp2(mw[ww][0] - m_all[nt][0]);
                        const float g1 = (mw[ww][1] == -INFINITY) ? 0.f : fast_exp2(mw[ww][1] - m_all[nt][1]);
                        l_all[nt][0] += lw[ww][0] * g0; l_all[nt][1] += lw[ww][1] * g1;
#pragma unroll
                        for (int a = 0; a < 8; ++a) {
                            const int d0 = 16 * a + rw;
                            o[nt][a][0] += g0 * sm.v.merge_o[ww][2 * qd][d0];
                            o[nt][a][1] += g1 * sm.v.merge_o[ww][2 * qd + 1][d0];
                            o[nt][a][2] += g0 * sm.v.merge_o[ww][2 * qd][d0 + 8];
                            o[nt][a][3] += g1 * sm.v.merge_o[ww][2 * qd + 1][d0 + 8];
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.merge_bar[1]);    // scratch may be refilled
                }
                ++seg;
            }
            if (w == 0) {
                const int u = mt.unit;
                const int n_held = sm.pieces_n;
                if (piece_tiles < mt.unit_tiles && n_held < kMaxPieces) {
                    // part of the unit: partial into the slot of the interval the piece began in
                    const size_t slot = (size_t)piece_iv + u;
                    float* po = p.part_o + slot * (8 * NT * kHeadDim);
                    float* pm = p.part_ml + slot * (kMlStride * NT);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const int c0 = 8 * nt + 2 * qd;
#pragma unroll
                        for (int a = 0; a < 8; ++a) {
                            const int d0 = 16 * a + rw;
                            po[c0 * kHeadDim + d0] = o[nt][a][0];
                            po[(c0 + 1) * kHeadDim + d0] = o[nt][a][1];
                            po[c0 * kHeadDim + d0 + 8] = o[nt][a][2];
                            po[(c0 + 1) * kHeadDim + d0 + 8] = o[nt][a][3];
                        }
                        if (rw == 0) {
                            pm[c0] = m_all[nt][0];
                            pm[c0 + 1] = m_all[nt][1];
                            pm[8 * NT + c0] = l_all[nt][0];
                            pm[8 * NT + c0 + 1] = l_all[nt][1];
                        }
                    }
                    if (lane == 0) {
                        pm[16 * NT] = __uint_as_float(p.generation);
                        sm.pieces_n = n_held + 1;
                    }
                    // Make the piece count at once (not at the end of the stream, which may be far off
                    // when this CTA goes on to take other ranges' chunks): the partial is made visible,
                    // then one 64-bit add on the unit's counter -- high half: tiles done; low half: one
                    // bit per piece, its slot's place among the unit's candidate slots, when there are at
                    // most 32 of those.  Lane k makes the add for the k-th piece held and keeps the
                    // answer in a register until the stream is over; nothing waits for it here.
                    __threadfence();
                    __syncwarp();
                    if (lane == n_held) {
                        const int iv_first = interval_of(sm.sched, mt.unit_first);
                        const int iv_last = interval_of(sm.sched, mt.unit_first + mt.unit_tiles - 1);
                        const int n_slots = iv_last - iv_first + 1;
                        const unsigned int bit = n_slots <= 32 ? 1u << (piece_iv - iv_first) : 0u;
                        sm.pieces[n_held] = Piece{u, piece_tiles, iv_first + u, n_slots, mt.unit_tiles};
                        tk_bit = bit;
                        tk_before = atomicAdd(&p.tickets[u], ((unsigned long long)piece_tiles << 32) | bit);
                    }
                    __syncwarp();
                } else if (piece_tiles >= mt.unit_tiles) {
                    // the whole unit in one piece: final output
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const int c0 = 8 * nt + 2 * qd;
                        const float inv0 = l_all[nt][0] > 0.f ? 1.f / l_all[nt][0] : 0.f;
                        const float inv1 = l_all[nt][1] > 0.f ? 1.f / l_all[nt][1] : 0.f;
                        const bool h0 = c0 < p.rows, h1 = c0 + 1 < p.rows;
                        const size_t row0 = unit_row(p, u, h0 ? c0 : 0), row1 = unit_row(p, u, h1 ? c0 + 1 : 0);
                        __nv_bfloat16* o0 = p.out + row0 * kHeadDim;
                        __nv_bfloat16* o1 = p.out + row1 * kHeadDim;
#pragma unroll
                        for (int a = 0; a < 8; ++a) {
                            const int d0 = 16 * a + rw;
                            if (h0) {
                                o0[d0] = __float2bfloat16(o[nt][a][0] * inv0);
                                o0[d0 + 8] = __float2bfloat16(o[nt][a][2] * inv0);
                            }
                            if (h1) {
                                o1[d0] = __float2bfloat16(o[nt][a][1] * inv1);
                                o1[d0 + 8] = __float2bfloat16(o[nt][a][3] * inv1);
                            }
                        }
                        if (p.lse && rw == 0) {
                            const float ln2 = 0.6931471805599453f;
                            if (h0) p.lse[row0] = l_all[nt][0] > 0.f ? (m_all[nt][0] + log2f(l_all[nt][0])) * ln2 : -INFINITY;
                            if (h1) p.lse[row1] = l_all[nt][1] > 0.f ? (m_all[nt][1] + log2f(l_all[nt][1])) * ln2 : -INFINITY;
                        }
                    }
                } else {
                    // (cannot happen with the schedule's bound on pieces per CTA) no room to hold
                    // the piece back: flag it rather than lose it silently
                    raise_status(p.status, DEV_TIMEOUT);
                }
            }
        }
        mt = nx;
    }
    } else {
    // ---------------- the unit's (17 to 64) rows on the MMA's M side, tokens on N ----------------
    // Warp w owns rows 16w .. 16w+15 of the unit and goes through all 64 tokens of every tile, so its
    // running max, sum and 16 x 128 output block are complete for its rows: nothing is folded across
    // warps when a piece ends.
    //     S (16 rows x 64 tok) = Q_w (16 x 128) . K^T (128 x 64)       mma.sync m16n8k16, K straight from its tile
    //     O (16 rows x 128)   += P (16 x 64) . V (64 x 128)           P from S's registers, V through ldmatrix.trans
    const int rA = 16 * w + rw, rB = rA + 8;                            // this thread's two rows
    const bool realA = rA < p.rows, realB = rB < p.rows;
    // newest cached tokens a row may not see (its query token's distance from the last one)
    const int backA = realA ? p.q_len - 1 - (p.t_base + ((rA * p.group_magic) >> 16)) : 0;
    const int backB = realB ? p.q_len - 1 - (p.t_base + ((rB * p.group_magic) >> 16)) : 0;
    uint32_t qa[8][4];                  // Q A-fragments: 8 k-steps over d
    float o[16][4];                     // O accumulators: 16 n-tiles of 8 channels
    float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;
    int pubs = 0;                       // partials written so far (phase of pub_bar)
    auto load_q_wide = [&](int unit) {
        const uint32_t* qrA = reinterpret_cast<const uint32_t*>(p.q + unit_row(p, unit, realA ? rA : 0) * kHeadDim);
        const uint32_t* qrB = reinterpret_cast<const uint32_t*>(p.q + unit_row(p, unit, realB ? rB : 0) * kHeadDim);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qa[ks][0] = realA ? __ldg(qrA + 8 * ks + qd) : 0u;
            qa[ks][1] = realB ? __ldg(qrB + 8 * ks + qd) : 0u;
            qa[ks][2] = realA ? __ldg(qrA + 8 * ks + 4 + qd) : 0u;
            qa[ks][3] = realB ? __ldg(qrB + 8 * ks + 4 + qd) : 0u;
        }
    };
    // lane-constant parts of the ldmatrix addresses (swizzle: 16-B chunk ^= row & 7)
    const int sw = lane & 7;
    const int k_cb = lane >> 3;                          // K: which of the four 8-channel blocks of a load
    const int v_tok = 8 * ((lane >> 3) & 1) + (lane & 7);  // V: token within a 16-token step
    const int v_cb = lane >> 4;                          // V: which of the two 8-channel blocks of a load
    if (!mbar_wait(&sm.full[0], 0, p.status)) return;
    if (tid == 0) SEER_STAMP(10);
    StageMeta mt = sm.meta[0];
    for (int it = 0; mt.nvalid >= 0; ++it) {
        const int st = it % kS;
        if (mt.flags & 1) {
            load_q_wide(mt.unit);
#pragma unroll
            for (int ct = 0; ct < 16; ++ct)
#pragma unroll
                for (int x = 0; x < 4; ++x) o[ct][x] = 0.f;
            mA = mB = -INFINITY;
            lA = lB = 0.f;
            piece_tiles = 0;
            piece_iv = mt.interval;
        }
        ++piece_tiles;
        const int nv = mt.nvalid;                          // cached tokens from the tile's first row on (capped at 64 + 7)
        if (nv > 0 && w * 16 < p.rows) {
            const uint32_t kbase = smem_u32(sm.stage[st]);
            const uint32_t vbase = kbase + kTileBytes;
            if (nv < kTileTokens) {
                // ragged tail: rows past the sequence end may hold anything; every warp clears them in V for
                // itself (the same zeros from all), so that 0-probability times garbage cannot produce NaN
                unsigned char* vt = sm.stage[st] + kTileBytes;
                for (int x = lane; x < (kTileTokens - nv) * 32; x += 32) {
                    const int r = nv + (x >> 5), part = x & 31;    // 32 x 8-byte pieces per row
                    const int half = part >> 4, off = (part & 15) * 8;
                    *reinterpret_cast<uint2*>(vt + half * kHalfTileBytes + r * 128 + off) = make_uint2(0u, 0u);
                }
                fence_proxy_async_smem();
                __syncwarp();
            }
            // The tile's 64 tokens are taken in two halves of 32, each a complete online-softmax step (scores,
            // running max and sum, P . V): half as many score and probability registers are live at a time.
            const int limA = nv - backA, limB = nv - backB;
#pragma unroll
            for (int hb = 0; hb < 2; ++hb) {
                if (32 * hb >= nv) break;                  // (nothing cached in the second half)
                // ---- S = Q . K^T ----
                float sc[4][4];
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) sc[jj][0] = sc[jj][1] = sc[jj][2] = sc[jj][3] = 0.f;
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int row = 8 * (4 * hb + jj) + (lane & 7);        // (row & 7 == lane & 7 == sw)
#pragma unroll
                    for (int kp = 0; kp < 4; ++kp) {
                        uint32_t b[4];
                        const int cb = 4 * kp + k_cb;      // 8-channel block 0..15
                        ldmatrix_x4(b, kbase + (cb >> 3) * kHalfTileBytes + row * 128 + (((cb & 7) ^ sw) << 4));
                        mma_bf16_16816(sc[jj], qa[2 * kp], b[0], b[1]);
                        mma_bf16_16816(sc[jj], qa[2 * kp + 1], b[2], b[3]);
                    }
                }
                // ---- mask, online softmax per row (a row's tokens sit in the four lanes of its quad) ----
                float mxA = -INFINITY, mxB = -INFINITY;
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int t0 = 8 * (4 * hb + jj) + 2 * qd;
                    sc[jj][0] = t0 < limA ? sc[jj][0] * p.scale_log2 : -INFINITY;
                    sc[jj][1] = t0 + 1 < limA ? sc[jj][1] * p.scale_log2 : -INFINITY;
                    sc[jj][2] = t0 < limB ? sc[jj][2] * p.scale_log2 : -INFINITY;
                    sc[jj][3] = t0 + 1 < limB ? sc[jj][3] * p.scale_log2 : -INFINITY;
                    mxA = fmaxf(mxA, fmaxf(sc[jj][0], sc[jj][1]));
                    mxB = fmaxf(mxB, fmaxf(sc[jj][2], sc[jj][3]));
                }
                mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 1));
                mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 1));
                mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 2));
                mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 2));
                const float mnA = fmaxf(mA, mxA), mnB = fmaxf(mB, mxB);
                // a row that has seen nothing so far keeps max = -inf; exponents are then taken against 0
                const float mbA = mnA == -INFINITY ? 0.f : mnA, mbB = mnB == -INFINITY ? 0.f : mnB;
                const float alA = fast_exp2(mA - mbA), alB = fast_exp2(mB - mbB);
                const bool same_max = __all_sync(0xffffffffu, mA == mnA && mB == mnB);
                mA = mnA; mB = mnB;
                float sumA = 0.f, sumB = 0.f;
                uint32_t pa[4][2];                         // P as bf16 pairs: [n-tile][row A | row B]
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const float p0 = fast_exp2(sc[jj][0] - mbA), p1 = fast_exp2(sc[jj][1] - mbA);
                    const float p2 = fast_exp2(sc[jj][2] - mbB), p3 = fast_exp2(sc[jj][3] - mbB);
                    sumA += p0 + p1;
                    sumB += p2 + p3;
                    pa[jj][0] = pack_bf16x2(p0, p1);
                    pa[jj][1] = pack_bf16x2(p2, p3);
                }
                lA = lA * alA + sumA;
                lB = lB * alB + sumB;
                if (!same_max) {
#pragma unroll
                    for (int ct = 0; ct < 16; ++ct) { o[ct][0] *= alA; o[ct][1] *= alA; o[ct][2] *= alB; o[ct][3] *= alB; }
                }
                // ---- O += P . V ----
#pragma unroll
                for (int k2 = 0; k2 < 2; ++k2) {
                    const uint32_t a[4] = {pa[2 * k2][0], pa[2 * k2][1], pa[2 * k2 + 1][0], pa[2 * k2 + 1][1]};
                    const int row = 16 * (2 * hb + k2) + v_tok;
#pragma unroll
                    for (int cp = 0; cp < 8; ++cp) {
                        uint32_t b[4];
                        const int cb = 2 * cp + v_cb;
                        ldmatrix_x4_trans(b, vbase + (cb >> 3) * kHalfTileBytes + row * 128 + (((cb & 7) ^ (row & 7)) << 4));
                        mma_bf16_16816(o[2 * cp], a, b[0], b[1]);
                        mma_bf16_16816(o[2 * cp + 1], a, b[2], b[3]);
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.empty[st]);

        // the next tile's metadata tells whether the piece goes on
        const int nst = (it + 1) % kS;
        if (!mbar_wait(&sm.full[nst], ((it + 1) / kS) & 1, p.status)) return;
        const StageMeta nx = sm.meta[nst];
        if (nx.flags & 1) {
            // ---------------- the current piece ends here: every warp stores its own rows -----------------
            float l0 = lA, l1 = lB;
            l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
            l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
            const int u = mt.unit;
            if (piece_tiles < mt.unit_tiles) {
                // part of the unit: partial into the slot of the interval the piece began in
                const size_t slot = (size_t)piece_iv + u;
                float* po = p.part_o + slot * (8 * NT * kHeadDim);
                float* pm = p.part_ml + slot * (kMlStride * NT);
#pragma unroll
                for (int ct = 0; ct < 16; ++ct) {
                    if (realA) *reinterpret_cast<float2*>(po + rA * kHeadDim + 8 * ct + 2 * qd) = make_float2(o[ct][0], o[ct][1]);
                    if (realB) *reinterpret_cast<float2*>(po + rB * kHeadDim + 8 * ct + 2 * qd) = make_float2(o[ct][2], o[ct][3]);
                }
                if (qd == 0) {
                    if (realA) { pm[rA] = mA; pm[8 * NT + rA] = l0; }
                    if (realB) { pm[rB] = mB; pm[8 * NT + rB] = l1; }
                }
                if (tid == 0) pm[16 * NT] = __uint_as_float(p.generation);
                // every warp makes its rows of the partial visible; then warp 0 counts the piece on the unit's
                // ticket (as in the other variant: lane k for the k-th piece held, answer kept in a register)
                __threadfence();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.merge_bar[0]);
                if (w == 0) {
                    if (!mbar_wait(&sm.merge_bar[0], pubs & 1, p.status)) return;
                    const int n_held = sm.pieces_n;
                    if (n_held < kMaxPieces) {
                        if (lane == n_held) {
                            const int iv_first = interval_of(sm.sched, mt.unit_first);
                            const int iv_last = interval_of(sm.sched, mt.unit_first + mt.unit_tiles - 1);
                            const int n_slots = iv_last - iv_first + 1;
                            const unsigned int bit = n_slots <= 32 ? 1u << (piece_iv - iv_first) : 0u;
                            sm.pieces[n_held] = Piece{u, piece_tiles, iv_first + u, n_slots, mt.unit_tiles};
                            tk_bit = bit;
                            tk_before = atomicAdd(&p.tickets[u], ((unsigned long long)piece_tiles << 32) | bit);
                        }
                        __syncwarp();
                        if (lane == 0) sm.pieces_n = n_held + 1;
                    } else {
                        raise_status(p.status, DEV_TIMEOUT);   // (cannot happen with the schedule's bound on pieces per CTA)
                    }
                }
                ++pubs;
            } else {
                // the whole unit in one piece: final output
                const float invA = l0 > 0.f ? 1.f / l0 : 0.f, invB = l1 > 0.f ? 1.f / l1 : 0.f;
                const size_t rowA = unit_row(p, u, realA ? rA : 0), rowB = unit_row(p, u, realB ? rB : 0);
                uint32_t* oA = reinterpret_cast<uint32_t*>(p.out + rowA * kHeadDim);
                uint32_t* oB = reinterpret_cast<uint32_t*>(p.out + rowB * kHeadDim);
#pragma unroll
                for (int ct = 0; ct < 16; ++ct) {
                    if (realA) oA[4 * ct + qd] = pack_bf16x2(o[ct][0] * invA, o[ct][1] * invA);
                    if (realB) oB[4 * ct + qd] = pack_bf16x2(o[ct][2] * invB, o[ct][3] * invB);
                }
                if (p.lse && qd == 0) {
                    const float ln2 = 0.6931471805599453f;
                    if (realA) p.lse[rowA] = l0 > 0.f ? (mA + log2f(l0)) * ln2 : -INFINITY;
                    if (realB) p.lse[rowB] = l1 > 0.f ? (mB + log2f(l1)) * ln2 : -INFINITY;
                }
            }
        }
        mt = nx;
    }
    }
    // ---- the stream is over: make this CTA's partials count, and do the combines it owes ------
    pdl_launch_dependents();
    if (tid == 0) SEER_STAMP(6);
    if (w == 0) {
        const int n_held = sm.pieces_n;
        // Every piece was added to its unit's counter when it ended.  Whoever completed a unit's tile
        // count learns from the same word which slots hold the unit's partials.
        if (lane == 0) SEER_STAMP(0);
        bool owe = false;
        Piece pc = Piece{0, 0, 0, 0, 0};
        int first_slot = 0, n_slots = 0;
        unsigned int mask = 0u;
        if (lane < n_held) {
            pc = sm.pieces[lane];                      // (unit, tiles, first slot, slots, tiles of the unit)
            first_slot = pc.unit_first;
            n_slots = pc.unit_tiles;
            owe = (int)(tk_before >> 32) + pc.tiles == pc.extra;     // this piece completed the unit's count
            mask = (unsigned int)tk_before | tk_bit;
        }
        // rewrite the list: the units this CTA has to combine, with their candidate slots
        const unsigned m = __ballot_sync(0xffffffffu, owe);
        __syncwarp();
        if (owe) {
            p.tickets[pc.unit] = 0ull;                 // ready for the next launch
            sm.pieces[__popc(m & ((1u << lane) - 1u))] = Piece{pc.unit, 0, first_slot, n_slots, (int)mask};
        }
        if (lane == 0) sm.pieces_n = __popc(m);
    }
    // every warp is done with the stage buffers, and warp 0's list of owed units is written
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.end_bar);
    if (!mbar_wait(&sm.end_bar, 0, p.status)) return;
    const int n_owed = sm.pieces_n;
    if (n_owed == 0) {                                 // nothing to combine: make room for the next kernel at once
        if (tid == 0) SEER_STAMP(7);
        return;
    }
#ifdef SEER_DECODE_TRACE
    if (tid == 0 && n_owed > 0) { SEER_STAMP(2); p.trace[(size_t)blockIdx.x * kTraceSlots + 4] = n_owed; }
#endif
    // The combines use the stage buffers as scratch (the stream is over, nothing is in flight).  Which
    // of a unit's candidate slots hold a partial of this launch is known from the start when the split
    // is static (all of them) or the unit has at most 32 candidates (the ticket word said which);
    // otherwise the four warps look at the generation stamps of a quarter of the candidates each and
    // list the valid ones in the third stage buffer.  Up to 2 * kDirect partials are added straight
    // from global memory; more are brought in by bulk copies, n_land at a time, into the first two
    // stage buffers (only the unit's real rows: rows x 512 B + 128 B * NT per partial, one per lane).
    constexpr int kSeg = kListInts / kConsumerWarps;             // slot numbers a warp can list per window
    int* lists = reinterpret_cast<int*>(sm.stage[SmemK::kBufs - 1]);   // [4][kSeg] slot numbers
    int* counts = lists + kListInts;                             // [4]
    constexpr int kMl = kMlStride * NT;                          // floats per (max, sum, stamp) record
    const int o_stride = p.rows * kHeadDim;                      // floats per staged partial
    // (the landing area is every stage buffer but the last: two of them, six in the tensor-memory variant)
    constexpr int kLand = (SmemK::kBufs - 1) * kStageBytes;
    const int n_land = min(32, kLand / (o_stride * 4 + kMl * 4));
    float* land_o = reinterpret_cast<float*>(sm.stage[0]);       // [n_land][rows][128]
    float* land_ml = land_o + n_land * o_stride;                 // [n_land][32 * NT]
    int sync_phase = 0, land_phase = 0;
    auto sync_consumers = [&]() -> bool {
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.list_bar);
        const bool ok = mbar_wait(&sm.list_bar, sync_phase & 1, p.status);
        ++sync_phase;
        return ok;
    };
    const bool all_valid = sm.sched.R == 0;
    bool lists_in_use = false;
#pragma unroll 1
    for (int e = 0; e < n_owed; ++e) {
        const int unit = sm.pieces[e].unit, first = sm.pieces[e].unit_first, n_slots = sm.pieces[e].unit_tiles;
        const unsigned int mask = (unsigned int)sm.pieces[e].extra;
        const bool by_mask = !all_valid && n_slots <= 32;
        MergeState<NT> ms;
        merge_init(ms);
#pragma unroll 1
        for (int w0 = 0; w0 < n_slots; w0 += kListInts) {
            const int win = min(kListInts, n_slots - w0);
            const bool listed = !all_valid && !by_mask;
            if (listed) {
                if (lists_in_use && !sync_consumers()) return;   // everybody is done with the previous lists
                lists_in_use = true;
                const int lo = w * kSeg, hi = min(win, lo + kSeg);
                const int n = lo < hi ? scan_valid_slots<NT>(p, first + w0 + lo, hi - lo, lists + lo, lane) : 0;
                if (lane == 0) counts[w] = n;
                if (!sync_consumers()) return;
            }
#pragma unroll 1
            for (int seg = 0; seg < (listed ? kConsumerWarps : 1); ++seg) {
                const int n = all_valid ? win : by_mask ? __popc(mask) : counts[seg];
                const int* seg_list = lists + seg * kSeg;
                if ((NT < kWideTiles || n_land < 2) && n <= 2 * kDirect) {
                    // up to two rounds of direct loads beat staging (one round trip each, no barrier); with the
                    // rows on M a thread's share of a partial is eight such round trips, and staging wins as
                    // long as more than one partial fits the landing area
                    unsigned int rem = mask;                 // bits of the valid slots not yet taken
#pragma unroll 1
                    for (int k0 = 0; k0 < n; k0 += kDirect) {
                        const int m = min(kDirect, n - k0);
                        int sl[kDirect];
#pragma unroll
                        for (int k = 0; k < kDirect; ++k) {
                            const int kk = k0 + min(k, m - 1);
                            if (by_mask) {
                                sl[k] = first + __ffs(rem) - 1;
                                if (k < m - 1) rem &= rem - 1;
                            } else {
                                sl[k] = all_valid ? first + w0 + kk : seg_list[kk];
                            }
                        }
                        if (by_mask) rem &= rem - 1;
                        merge_accumulate_direct<NT>(p, ms, sl, m, tid);
                    }
                    continue;
                }
                // the k-th valid slot of this segment
                auto slot_at = [&](int k) -> int {
                    return all_valid ? first + w0 + k : by_mask ? first + (int)__fns(mask, 0u, k + 1) : seg_list[k];
                };
#pragma unroll 1
                for (int s0 = 0; s0 < n; s0 += n_land) {
                    const int m = min(n_land, n - s0);
                    if (w == 0) {
                        // warp 0 issues the copies, one partial per lane
                        if (lane == 0) {
                            fence_proxy_async_smem();        // earlier plain accesses to the landing area are done
                            mbar_arrive_expect_tx(&sm.land_bar, (uint32_t)m * (o_stride * 4 + kMl * 4));
                        }
                        __syncwarp();
                        if (lane < m) {
                            const size_t sl = (size_t)slot_at(s0 + lane);
                            bulk_load(land_o + lane * o_stride, p.part_o + sl * (8 * NT * kHeadDim), o_stride * 4, &sm.land_bar);
                            bulk_load(land_ml + lane * kMl, p.part_ml + sl * kMl, kMl * 4, &sm.land_bar);
                        }
                    }
                    if (!mbar_wait(&sm.land_bar, land_phase & 1, p.status)) return;
#ifdef SEER_DECODE_TRACE
                    if (tid == 0 && land_phase == 0) SEER_STAMP(5);
#endif
                    ++land_phase;
                    merge_accumulate_staged<NT>(ms, land_o, o_stride, land_ml, m, p.rows, tid);
                    if (!sync_consumers()) return;           // everybody has read the landing area
                }
            }
        }
        merge_finalize(p, ms, unit, tid);
    }
    if (tid == 0) SEER_STAMP(7);
}

template <bool TC>
constexpr size_t decode_smem_bytes() { return sizeof(SmemT<TC>) + 1024; }

template <bool SPARSE, bool PAGED, int NT, bool SMALL, bool TC = false>
cudaError_t configure() {
    return cudaFuncSetAttribute(decode_kernel<SPARSE, PAGED, NT, SMALL, TC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)decode_smem_bytes<TC>());
}

template <bool SPARSE, bool PAGED, int NT, bool SMALL, bool TC = false>
int occupancy() {
    static int cached[kMaxDevices] = {};             // 0: not asked yet on that device
    const int slot = current_device_slot();
    if (cached[slot] <= 0) {
        if (configure<SPARSE, PAGED, NT, SMALL, TC>() != cudaSuccess) return 0;
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_kernel<SPARSE, PAGED, NT, SMALL, TC>,
                                                          TC ? kTcThreads : kThreads, decode_smem_bytes<TC>()) != cudaSuccess)
            return 0;
        cached[slot] = n;
    }
    return cached[slot];
}

template <bool SPARSE, bool PAGED, int NT, bool SMALL, bool TC = false>
cudaError_t launch(const CUtensorMap& mk, const CUtensorMap& mv, const DecodeParams& p, int grid,
                   cudaStream_t stream) {
    if (occupancy<SPARSE, PAGED, NT, SMALL, TC>() <= 0) return cudaErrorInvalidConfiguration;
    return launch_pdl(decode_kernel<SPARSE, PAGED, NT, SMALL, TC>, dim3(grid), dim3(TC ? kTcThreads : kThreads),
                      decode_smem_bytes<TC>(), stream, mk, mv, p);
}

// (blocks of 16 or 32 tokens use the same resources: the occupancy of the 64-token variant stands for both)
template <int NT, bool TC = false>
int occupancy_of(bool sparse, bool paged) {
    if (sparse) return paged ? occupancy<true, true, NT, false, TC>() : occupancy<true, false, NT, false, TC>();
    return paged ? occupancy<false, true, NT, false, TC>() : occupancy<false, false, NT, false, TC>();
}

template <int NT, bool TC = false>
cudaError_t launch_of(bool sparse, bool paged, const CUtensorMap& map_k, const CUtensorMap& map_v,
                      const DecodeParams& p, int grid, cudaStream_t stream) {
    if constexpr (NT < kWideTiles) {            // (the rows-on-M variants take blocks of 64 or 128 tokens only)
        if (sparse && p.blocks_per_tile > 1)
            return paged ? launch<true, true, NT, true>(map_k, map_v, p, grid, stream)
                         : launch<true, false, NT, true>(map_k, map_v, p, grid, stream);
    }
    if (sparse) return paged ? launch<true, true, NT, false, TC>(map_k, map_v, p, grid, stream)
                             : launch<true, false, NT, false, TC>(map_k, map_v, p, grid, stream);
    return paged ? launch<false, true, NT, false, TC>(map_k, map_v, p, grid, stream)
                 : launch<false, false, NT, false, TC>(map_k, map_v, p, grid, stream);
}

}  // namespace

// n_tiles: 1 or 2 (the unit's rows on the MMA's N side), 8 (rows on M, mma.sync), 16 (rows on M, tcgen05:
// the same 64-row partial slots as 8)
int decode_ctas_per_sm(bool sparse, bool paged, int n_tiles) {
    return n_tiles == 1   ? occupancy_of<1>(sparse, paged)
           : n_tiles == 2 ? occupancy_of<2>(sparse, paged)
           : n_tiles == kTcTilesCode ? occupancy_of<kWideTiles, true>(sparse, paged)
                                     : occupancy_of<kWideTiles>(sparse, paged);
}

int decode_max_intervals(int grid, int max_rounds) { return grid * (max_rounds + 1) + 1; }

cudaError_t launch_decode(bool sparse, bool paged, int n_tiles, const CUtensorMap& map_k, const CUtensorMap& map_v,
                          const DecodeParams& p, int grid, cudaStream_t stream) {
    const int slot_tiles = n_tiles == kTcTilesCode ? kWideTiles : n_tiles;
    if ((n_tiles != 1 && n_tiles != 2 && n_tiles != kWideTiles && n_tiles != kTcTilesCode) || p.rows > 8 * slot_tiles)
        return cudaErrorInvalidValue;
    if (slot_tiles == kWideTiles && p.blocks_per_tile > 1) return cudaErrorInvalidValue;
    return n_tiles == 1   ? launch_of<1>(sparse, paged, map_k, map_v, p, grid, stream)
           : n_tiles == 2 ? launch_of<2>(sparse, paged, map_k, map_v, p, grid, stream)
           : n_tiles == kTcTilesCode ? launch_of<kWideTiles, true>(sparse, paged, map_k, map_v, p, grid, stream)
                                     : launch_of<kWideTiles>(sparse, paged, map_k, map_v, p, grid, stream);
}

}  // namespace seer
