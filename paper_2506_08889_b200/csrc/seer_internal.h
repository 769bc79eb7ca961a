// Host-side declarations shared by the translation units of the library.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace seer {

constexpr int kHeadDim = 128;       // d
constexpr int kTileTokens = 64;     // tokens per staged K (or V) tile
constexpr int kMaxGroup = 8;        // query heads per KV head handled by one MMA N-tile
constexpr int kMaxDGate = 256;      // gate width: 64, 128 or 256
constexpr int kMaxRounds = 12;      // halving rounds of the decode kernels' dynamic tile pool

// Kernel attributes (the opt-in to more dynamic shared memory) are per device: index of the current
// device into per-device "already configured" tables (processes here use one GPU, the library does
// not assume it).
constexpr int kMaxDevices = 64;
inline int current_device_slot() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) dev = 0;
    return dev % kMaxDevices;
}

// Launch with the programmatic-stream-serialisation attribute (see pdl_wait in seer_device.cuh).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Everything the decode kernels need besides the two tensor maps.
struct DecodeParams {
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    float* lse;
    const int32_t* seq_lens;
    const int32_t* block_idx;       // sparse only
    const int32_t* block_cnt;       // sparse only, may be null
    const int32_t* page_table;      // paged only
    int64_t page_table_stride;
    int max_sel;
    int page_size;
    int num_pages;
    int batch, num_q_heads, num_kv_heads, group, block_size, tiles_per_block;
    int blocks_per_tile;            // 64 / block_size for blocks of 16 or 32 tokens (a tile gathers several listed blocks), else 1
    int bs_shift, tpb_shift, bpt_shift;   // log2 of block_size, tiles_per_block, blocks_per_tile
    unsigned int kvh_magic;         // ceil(2^32 / num_kv_heads), 0 for one KV head: unit / num_kv_heads by __umulhi
    int group_magic;                // ceil(2^16 / group): r / group = (r * group_magic) >> 16 for r < 16
    int q_len;                      // query tokens per sequence (the last q_len cached tokens), 1 for plain decoding
    int t_base, t_cnt;              // this launch handles query tokens t_base .. t_base + t_cnt - 1
    int rows;                       // t_cnt * group: rows on the MMA N side, <= 8 * (N-tiles of the kernel)
    int num_units;                  // batch * num_kv_heads
    int max_blocks_cap;             // tile-count clamp for dense: capacity in tiles
    int pool_div;                   // 1/pool_div of the tiles are handed out dynamically (0: none)
    int min_tiles;                  // a CTA's range has at least this many tiles (fewer CTAs take part when work is short)
    int max_rounds;                 // most dynamic chunks per range (<= kMaxRounds; 0: none) -- bounds the partial slots
    float scale_log2;               // sm_scale * log2(e)
    const int* list_flags;          // non-null: unit u's list is final once list_flags[u] == list_gen (written by the gate
    int list_gen;                   // kernel of the same step); the producer warp then waits per unit, not for the gate's grid
    int sel_from_lens;              // > 0: every unit's list holds min(this, blocks of its sequence) entries, so the
                                    // counts follow from the lengths and the schedule can be made before the kernel
                                    // that writes the lists has finished (0: read block_cnt)
    unsigned int* status;
    unsigned long long* tickets;    // [num_units]: tiles done << 32 | valid-slot bits; zero between launches
    int* sched;                     // [2]: theft cursor, exit counter; zero between launches
    int* steal;                     // [grid]: per-range claim counters (front | back << 16); zero between launches
    unsigned int generation;        // stamp that marks this launch's partials
    int* prefix;                    // [num_units + 1] prefix sums of the units' tile counts
    float* part_o;                  // [slots][8*NT][128]   (NT: N-tiles of the kernel, 1 or 2)
    float* part_ml;                 // [slots][32*NT]: max[8*NT], sum[8*NT], generation stamp
#ifdef SEER_DECODE_TRACE
    unsigned long long* trace;      // [grid][8] %globaltimer stamps (diagnostic builds only)
#endif
};

struct DecodeLaunch {
    int grid;
    cudaStream_t stream;
};

// Returns resident CTAs per SM for the decode kernel (queried once).
int decode_ctas_per_sm(bool sparse, bool paged, int n_tiles);
// Upper bound on the number of work intervals (static ranges + dynamic chunks) of a launch.
int decode_max_intervals(int grid, int max_rounds = kMaxRounds);
// n_tiles: MMA N-tiles of 8 rows (1 or 2: tokens on M), or 8 for the variant with the unit's (up to 64) rows on M;
// p.rows <= 8 * n_tiles.
cudaError_t launch_decode(bool sparse, bool paged, int n_tiles, const CUtensorMap& map_k, const CUtensorMap& map_v,
                          const DecodeParams& p, int grid, cudaStream_t stream);

struct GateParams {
    const __nv_bfloat16* q_nope;    // [B,Hq,d]
    const __nv_bfloat16* w_q;       // [Hkv,dg,g*d]
    const __nv_bfloat16* kcomp;     // [B,Hkv,max_blocks,dg]
    const int32_t* seq_lens;
    const float* scores_in;         // may be null
    float* scores;                  // [B,Hkv,max_blocks] (workspace or caller's scores_out)
    float* scores_user;             // caller's scores_out or null
    float* q_gate;                  // [B,Hkv,dg] workspace
    int32_t* block_idx;
    int32_t* block_cnt;
    int batch, num_q_heads, num_kv_heads, group, block_size;
    int d_gate, max_blocks, max_sel, token_budget;
    int q_len;                      // query tokens per sequence (1 for plain decoding); q_nope is [B,q_len,Hq,d]
    int threshold_mode;             // 0: token budget, 1: softmax probability above `threshold`
    float threshold;
    unsigned int* status;
    int* tickets;                   // [B*Hkv], zero between launches
    int* list_flags;                // non-null: list_gen is stored (release) to list_flags[u] once unit u's list is written
    int list_gen;
    double inv_freq[kMaxDGate / 2]; // rope_theta^(-2c/d_gate), computed on the host in double
};
// Launches the scoring kernels (unless scores_in is given) and the selection kernel.
// Returns the number of kernels launched through *launched.
cudaError_t launch_gate_select(const GateParams& p, cudaStream_t stream, int* launched);
// Whether a gate over max_blocks compressed keys per unit runs as the one cluster kernel (the only
// path that takes several query tokens).
bool gate_one_kernel(int max_blocks);

struct KcompParams {
    const __nv_bfloat16* k_nope;
    const __nv_bfloat16* w_k;       // [Hkv,dg,3d]
    __nv_bfloat16* kcomp;           // [B,Hkv,max_blocks,dg]
    const int32_t* seq_lens;
    int64_t stride_batch, stride_head, stride_token;
    int rows_block_local;
    int first_block, num_blocks;    // first_block == -t (1..8): the block that filled while the last t tokens were appended
    int wait_at_end;                // append only: work first, wait for the preceding kernel just before the end
    int batch, num_kv_heads, block_size, d_gate, max_blocks;
    int sm_count;                   // bulk build: one persistent CTA per SM
    unsigned int* status;           // sticky device status word (bounded waits report here)
#ifdef SEER_DECODE_TRACE
    unsigned long long* trace;      // diagnostic builds: per-warp cycle counters of the bulk build
#endif
    double inv_freq[kMaxDGate / 2];
};
// True when the bulk build of these parameters runs as the persistent streaming kernel, which reads the keys
// through a tensor map (channel, token row, head, sequence) with a box of 64 channels x kKcompStageRows rows,
// 128-byte swizzle; launch_kcomp_append falls back to the plain-load kernel when it is given no map.
constexpr int kKcompStageRows = 64;
bool kcomp_bulk_streams(const KcompParams& p);
cudaError_t launch_kcomp_append(const KcompParams& p, const CUtensorMap* map_k, cudaStream_t stream, int* launched);

}  // namespace seer
