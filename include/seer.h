/*
 * seer.h -- C ABI of the B200 (sm_100a) decode library for SeerAttention-R:
 * AttnGate scoring over a K compression cache, token-budget block selection,
 * block-sparse GQA split-KV flash decoding with a log-sum-exp combine, the
 * compressed-K cache update, and a dense decode kernel of the same design.
 *
 * General rules
 *  - Every tensor pointer is a DEVICE pointer owned by the caller, unless a
 *    comment says "host".  The structs themselves are read on the host.
 *  - bf16 tensors are raw 16-bit bfloat16; strides are in ELEMENTS.
 *  - Every entry point is asynchronous on the CUDA stream passed as
 *    `stream` (a cudaStream_t cast to void*, NULL = default stream), performs
 *    no host synchronisation and no device allocation.  The library allocates
 *    device memory only in seer_create (context workspace).
 *  - Errors that the host can see (null pointers, unsupported shapes, a too
 *    small workspace) return a status at once and launch nothing.  Problems
 *    only the device can see (a block index or page id out of range) never
 *    trap: the entry is skipped and a sticky flag is raised that
 *    seer_get_device_status reports.
 *  - A context serialises its calls through its workspace: calls that share a
 *    context must be ordered on one stream (or by events).  Use one context
 *    per concurrent stream.
 *  - Supported: head_dim 128; block_size 16, 32, 64 or 128 (the range of the
 *    paper's block-size study, Sec. 5 "Block Size for Sparse Attention"; 64 is
 *    its default); group size num_q_heads / num_kv_heads in 1..8; bf16 inputs,
 *    fp32 accumulation.
 *
 * Notation: B batch, Hq query heads, Hkv KV heads, g = Hq / Hkv, d head_dim,
 * b block_size, L_i KV length of sequence i INCLUDING the token being decoded,
 * n_i = ceil(L_i / b) blocks.  Query head hq belongs to KV head hq / g.
 */
#ifndef SEER_H_
#define SEER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct seer_ctx seer_ctx;

typedef enum {
    SEER_OK = 0,
    SEER_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, bad stride/alignment */
    SEER_ERR_UNSUPPORTED = 2,   /* shape outside the supported set listed above */
    SEER_ERR_WORKSPACE = 3,     /* context workspace too small for this call */
    SEER_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed (see seer_last_error) */
    SEER_ERR_BAD_INDEX = 5,     /* device saw a block index / page id out of range (skipped) */
    SEER_ERR_TIMEOUT = 6        /* a bounded device-side wait gave up (results invalid) */
} seer_status;

/* Problem shape shared by all calls. */
typedef struct {
    int batch;          /* B */
    int num_q_heads;    /* Hq */
    int num_kv_heads;   /* Hkv, divides Hq */
    int head_dim;       /* d = 128 */
    int block_size;     /* b = 16, 32, 64 or 128 (sparsity block of the gate, Sec. 2.2 / 3.1) */
    float sm_scale;     /* softmax scale applied to <q,k>, e.g. 1/sqrt(d) */
} seer_shape;

/*
 * bf16 K/V cache.  Two layouts:
 *  contiguous (page_table == NULL): element (i, h, t, c) of K is at
 *      k[i*stride_batch + h*stride_head + t*stride_token + c], t < max_seq_len.
 *      Any order of the batch/head/token axes works ([B,Hkv,S,d], [B,S,Hkv,d] ...).
 *  paged (page_table != NULL): the cache is a pool of num_pages pages of
 *      page_size tokens; token t of sequence i lives in page
 *      p = page_table[i*page_table_stride + t/page_size] at
 *      k[p*stride_batch + h*stride_head + (t % page_size)*stride_token + c].
 *      page_size must be a multiple of 64.  (The paper leaves paged KV to
 *      future work, Sec. 6; this layout is the library's own.)
 * All strides must be multiples of 8 elements and k, v 16-byte aligned.
 * Rows at positions >= L_i may hold anything (they are masked, never used).
 */
typedef struct {
    const void* k;
    const void* v;
    int64_t stride_batch;           /* between sequences, or between pages when paged */
    int64_t stride_head;
    int64_t stride_token;
    const int32_t* page_table;      /* device, or NULL for the contiguous layout */
    int64_t page_table_stride;      /* entries per sequence row of the page table */
    int page_size;                  /* tokens per page (paged only) */
    int num_pages;                  /* pages in the pool (paged only) */
    const int32_t* seq_lens;        /* device [B]: L_i */
    int max_seq_len;                /* token capacity per sequence (contiguous) or the
                                       largest L_i the page table covers (paged) */
} seer_kv;

/*
 * AttnGate parameters and the K compression cache (Eq. 1, Sec. 3.2).
 *  w_q   [Hkv, d_gate, g*d]  bf16: one projection per KV head over the g
 *        pre-RoPE query heads of its group laid end to end (index u*d + c).
 *  w_k   [Hkv, d_gate, 3*d]  bf16: input order [max-pool | min-pool | avg-pool].
 *  kcomp [B, Hkv, max_blocks, d_gate] bf16: entry j is the compressed key of
 *        block j (after pooling, projection and RoPE at position j*b).
 * RoPE inside the gate: rotate-half pairing (c, c + d_gate/2), angle
 * pos * rope_theta^(-2c/d_gate).  d_gate is 64, 128 or 256.
 */
typedef struct {
    int d_gate;
    float rope_theta;
    const void* w_q;
    const void* w_k;
    void* kcomp;
    int max_blocks;
} seer_gate;

/* ---- context ----------------------------------------------------------- */

/* Creates a context on CUDA device `device` and allocates its workspace
 * (workspace_bytes, 0 = a default of 64 MiB; partial results of split
 * sequences, gate scratch, status words).  *out is NULL on failure.
 * Read from the environment at creation: SEER_DECODE_WIDE_VARIANT and
 * SEER_STEP_LIST_FLAGS (the latter under seer_decode_step); read at the
 * process's first gate call: SEER_GATE_WIDEN (0: the gate's clusters keep one
 * CTA per 512 compressed keys also when there are few sequences; n: they may be
 * widened while all of them fit the SMs at n CTAs each, default 2).  Also at
 * creation, for experiments with the decode kernel's work split:
 * SEER_DECODE_POOL_DIV (1/n of a CTA's tiles are handed out dynamically;
 * default 4, 0 = a static split) and SEER_DECODE_MIN_TILES (fewest tiles a CTA
 * takes when work is short; default 4).  The
 * multi-token decode calls with 17 to 64 rows per (sequence, KV head)
 * (q_len * group) have two kernels: 16 = on the tcgen05 tensor cores with S, P,
 * O and the queries in tensor memory, 8 = mma.sync.  Unset, up to 48 rows take
 * the first and more rows the second (the faster one each, as measured).
 * Results agree within the decode tolerance. */
seer_status seer_create(seer_ctx** out, int device, size_t workspace_bytes);
/* Frees the workspace.  The caller must have synchronised the streams used. */
void seer_destroy(seer_ctx* ctx);
const char* seer_status_string(seer_status s);
/* Human-readable detail of the last failing call on this context (host string,
 * owned by the context, valid until the next call). */
const char* seer_last_error(const seer_ctx* ctx);
/* Synchronises `stream`, returns the sticky device-side status (SEER_OK,
 * SEER_ERR_BAD_INDEX or SEER_ERR_TIMEOUT) and clears it.  After SEER_ERR_TIMEOUT the
 * results of the calls since the last check are invalid; the context's counters are
 * reset by this call and the context can be used again. */
seer_status seer_get_device_status(seer_ctx* ctx, void* stream);

/*
 * Diagnostic: exercises the path every bounded device-side wait of the library takes when it runs out
 * (the waits are on a kernel's own copies in flight and, inside seer_decode_step, on the marks that the gate
 * kernel launched just before it leaves for each finished list).
 * One CTA polls `polls` times (1 .. 2^20) on a barrier that nobody arrives at, gives up, sets the sticky
 * time-out bit and leaves a ticket and the scheduler counters non-zero, as a kernel that was cut short
 * would.  The next seer_get_device_status then returns SEER_ERR_TIMEOUT and clears those counters, after
 * which the context works as before.  Asynchronous on `stream`; faults nothing.
 */
seer_status seer_debug_wait_timeout(seer_ctx* ctx, int polls, void* stream);
/*
 * Diagnostic for the roofline (the paper's kernel is "primarily I/O-bound", Sec. 4.4: its ceiling is what a
 * kernel that only reads gets out of the memory): reads `bytes` bytes at `src` once -- device memory,
 * 16-byte aligned, `bytes` a multiple of 16 -- with plain 16-byte loads, eight in flight per thread, and
 * leaves the exclusive-or of all their 32-bit words in the low half of *checksum (device memory, 8 bytes,
 * cleared by the call).  Timed by the caller over a buffer larger than the L2 cache it gives the read
 * bandwidth that the decode kernels' achieved figures can be set against.  Asynchronous on `stream`.
 */
seer_status seer_debug_read_bandwidth(seer_ctx* ctx, const void* src, size_t bytes, unsigned long long* checksum,
                                      void* stream);
/* Workspace bytes a context needs for calls of this shape (upper bound);
 * max_blocks = largest number of blocks per sequence. */
size_t seer_workspace_bytes(const seer_shape* shape, int max_blocks, int d_gate);
/* Number of kernels launched by this context so far (all entry points). */
uint64_t seer_launch_count(const seer_ctx* ctx);

/* ---- the four operations ------------------------------------------------ */

/*
 * Dense decode attention (the baseline of the paper's kernel comparison,
 * Sec. 4.4, here the library's own kernel): for every sequence i and query
 * head hq,  out[i,hq,:] = sum_{t < L_i} softmax_t(sm_scale <q[i,hq], k[i,hq/g,t]>) v[i,hq/g,t].
 *  q   [B,Hq,d] bf16 contiguous;  out [B,Hq,d] bf16 contiguous;
 *  lse [B,Hq] fp32 or NULL: natural-log sum of exp of the scaled scores.
 * L_i == 0 gives out = 0, lse = -inf.
 */
seer_status seer_dense_decode(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv,
                              const void* q, void* out, float* lse, void* stream);
/* Stream capture: the decode calls (dense, sparse, their _multi forms and the step calls) give every launch
 * counters that the host advances per call, so a CUDA graph captured from them could not be replayed
 * correctly; on a stream that is being captured they return SEER_ERR_UNSUPPORTED and enqueue nothing. */

/*
 * Block-sparse split-KV flash decoding (Sec. 3.3): the same sum restricted to
 * the tokens of the selected blocks, t in [j*b, min((j+1)*b, L_i)) for j in
 * the list of (i, hq/g); all query heads of a group share the list.
 *  block_idx [B,Hkv,max_sel] int32: block numbers; negative entries are
 *            padding and are skipped; entries >= n_i are skipped and raise
 *            SEER_ERR_BAD_INDEX; repeated entries are a caller error
 *            (the block would be counted twice).  Any order.
 *  block_cnt [B,Hkv] int32 or NULL: number of leading entries to read per
 *            list (NULL = all max_sel entries, relying on negative padding).
 * The selected blocks of all (sequence, KV head) pairs are cut into 64-token
 * tiles and dealt out evenly over the CTAs; pieces of one pair meet in a
 * log-sum-exp combine done by the last CTA to finish (no second launch).
 * A list with no valid entry gives out = 0, lse = -inf.
 * block_idx, block_cnt and seq_lens may be written by the kernel launched just
 * before this call on the stream: they are read only once that kernel has completed.
 */
seer_status seer_sparse_decode(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv,
                               const void* q, const int32_t* block_idx,
                               const int32_t* block_cnt, int max_sel,
                               void* out, float* lse, void* stream);

/*
 * The same two kernels for q_len query tokens per sequence (1 <= q_len <= 8): the query-level
 * parallelism of multi-token prediction or speculative decoding that Sec. 6 ("Unify Sparse
 * Prefill and Decoding") names as a way to more parallelism in sparse decoding.  The paper gives
 * no formula; this library takes the causal definition.  The cache already holds all L_i tokens
 * of sequence i, the newest q_len of them being the queries' own; query t (0 <= t < q_len) sits
 * at position L_i - q_len + t and sees cached tokens at positions <= its own -- for the sparse
 * call, of the blocks in the list of its (sequence, KV head), one list serving all q_len tokens
 * as it serves all heads of the group.  q_len = 1 is seer_sparse_decode / seer_dense_decode.
 *  q   [B,q_len,Hq,d] bf16 contiguous;  out [B,q_len,Hq,d] bf16;  lse [B,q_len,Hq] fp32 or NULL.
 * A query that sees no listed token (also every query at a negative position, when
 * L_i < q_len) gets out = 0, lse = -inf.  All tokens share one launch -- and the selected K/V
 * are read once for all of them -- while q_len * (Hq/Hkv) <= 64 (with blocks of 16 or 32 tokens:
 * <= 16); beyond that the call issues one launch per 64 (16) rows on the stream.  Other
 * arguments, errors and the treatment of the lists as in the single-token calls.
 */
seer_status seer_sparse_decode_multi(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv,
                                     const void* q, int q_len, const int32_t* block_idx,
                                     const int32_t* block_cnt, int max_sel, void* out, float* lse,
                                     void* stream);
seer_status seer_dense_decode_multi(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv,
                                    const void* q, int q_len, void* out, float* lse, void* stream);

/*
 * AttnGate scoring and token-budget selection (Eq. 1a, 1c; Sec. 3.1, 3.2).
 *  Scores: q_gate = RoPE_{pos = L_i-1}(w_q[h] x), score[j] = <q_gate, kcomp[i,h,j]> / sqrt(d_gate)
 *  for the blocks j < n_i - 1 (the softmax of Eq. 1c is not needed for a
 *  top-k decision and is not computed).
 *  Selection: k = min(max(1, token_budget / b), n_i, max_sel); the last block
 *  n_i - 1 is always selected and counts against k; the other k-1 are the
 *  highest-scoring of blocks [0, n_i-1), ties broken towards the lower block
 *  number (-0 == +0, NaN below every number).  Lists are written in ascending
 *  block order and padded with -1.
 *  q_nope    [B,Hq,d] bf16 pre-RoPE queries; may be NULL iff scores_in is given.
 *  scores_in [B,Hkv,max_blocks] fp32 or NULL: use these scores instead of
 *            computing them (selection on caller-provided scores).
 *  scores_out[B,Hkv,max_blocks] fp32 or NULL: receives the computed scores.
 *  block_idx [B,Hkv,max_sel] int32 out; block_cnt [B,Hkv] int32 out.
 *  seq_lens  device [B].
 */
seer_status seer_gate_select(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate,
                             const int32_t* seq_lens, const void* q_nope,
                             const float* scores_in, int token_budget,
                             int32_t* block_idx, int32_t* block_cnt, int max_sel,
                             float* scores_out, void* stream);

/*
 * The gate for q_len query tokens per sequence (the newest q_len cached tokens, as in
 * seer_sparse_decode_multi), producing the one block list per (sequence, KV head) that the
 * multi-token decode takes.  The paper has no gate for several decode-time queries (Sec. 6 only
 * names the direction); this library's reading: every query token t gets its own gate query,
 * rotated at its own position L_i - q_len + t (Eq. 1a); a block's score is the largest of the
 * q_len tokens' scores (Eq. 1c without the softmax), over the blocks that lie wholly before the
 * first query token, j < j_f = floor((L_i - q_len) / b); the blocks that hold a query token's own
 * position, j_f .. n_i - 1 (one or two), are always selected and count against the budget;
 * the other min(max(1, budget/b), n_i, max_sel) - (n_i - j_f) come from [0, j_f) by (score
 * descending, index ascending).  q_len = 1 is seer_gate_select.
 *  q_nope [B,q_len,Hq,d] bf16 (ignored when scores_in is given: selection only, scores_in holding
 *  the per-block maxima).  1 <= q_len <= 8.
 * Other arguments, outputs and errors as in seer_gate_select.
 */
seer_status seer_gate_select_multi(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate,
                                   const int32_t* seq_lens, const void* q_nope, const float* scores_in,
                                   int q_len, int token_budget, int32_t* block_idx, int32_t* block_cnt,
                                   int max_sel, float* scores_out, void* stream);

/*
 * The threshold method (Sec. 3.1, second method) for q_len query tokens per sequence.  The paper has
 * neither; the reading combines the two above: the per-block scores are the maxima over the tokens'
 * scores, the softmax runs over the candidate blocks [0, j_f), a candidate is selected when its
 * probability exceeds `threshold`, the blocks j_f .. n_i - 1 that hold the query tokens are always
 * selected and take no part in the normalisation, and when more candidates pass than max_sel leaves room
 * for beside those, the highest-scoring ones are kept.  q_len = 1 is seer_gate_select_threshold.
 * Arguments as in seer_gate_select_multi (threshold in [0, 1] in place of the token budget).
 */
seer_status seer_gate_select_threshold_multi(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate,
                                             const int32_t* seq_lens, const void* q_nope, const float* scores_in,
                                             int q_len, float threshold, int32_t* block_idx, int32_t* block_cnt,
                                             int max_sel, float* scores_out, void* stream);

/*
 * The threshold method of Sec. 3.1: the scores are normalised by a softmax over the blocks
 * that have a compressed key (Eq. 1c; blocks [0, n_i - 1)), and the blocks whose probability
 * exceeds `threshold` are selected -- a different number for every (sequence, KV head).  The
 * last block is always selected and takes no part in the normalisation; if more than
 * max_sel - 1 blocks pass, the max_sel - 1 highest-scoring are kept.  Scores must be finite.
 * The probabilities are formed in fp32, so a block whose probability is within rounding of
 * the threshold may fall on either side.  Other arguments and the output format as for
 * seer_gate_select (threshold in [0, 1]; the paper's ablation uses 2e-3 .. 6e-3).
 */
seer_status seer_gate_select_threshold(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate,
                                       const int32_t* seq_lens, const void* q_nope, const float* scores_in,
                                       float threshold, int32_t* block_idx, int32_t* block_cnt, int max_sel,
                                       float* scores_out, void* stream);

/*
 * K compression cache update (Eq. 1b; Sec. 2.2 "Pooling-based Compression of
 * K", Sec. 3.2): for block j of (i, h): per channel max, min and mean over the
 * block's b rows of pre-RoPE K, concatenated [max|min|avg], multiplied by
 * w_k[h], rotated at position j*b, stored as bf16 in kcomp[i,h,j,:].
 *  k_nope: bf16, row for token t of (i,h) at
 *          k_nope[i*stride_batch + h*stride_head + r*stride_token + c] with
 *          r = t (rows_block_local == 0) or r = t - j*b (rows_block_local != 0:
 *          the buffer holds just the block being appended, e.g. a rolling
 *          window of the last b tokens).
 *  first_block >= 0: write blocks first_block .. first_block+num_blocks-1 of
 *          every sequence, skipping blocks that are not complete
 *          (j >= floor(L_i / b)) -- the bulk build after prefill.
 *  first_block == -1: per sequence, write the block that has just filled,
 *          j = L_i/b - 1, if L_i % b == 0 and L_i > 0; otherwise nothing
 *          (num_blocks is ignored) -- the once-per-b-tokens update of decoding.
 *  first_block == -t, 2 <= t <= 8: the same after t tokens were appended at once
 *          (multi-token decoding): block j = floor(L_i/b) - 1 is written if its last
 *          row is among the t newest tokens, i.e. L_i >= b and L_i % b < t.
 */
seer_status seer_kcomp_append(seer_ctx* ctx, const seer_shape* shape, const seer_gate* gate,
                              const int32_t* seq_lens, const void* k_nope,
                              int64_t stride_batch, int64_t stride_head, int64_t stride_token,
                              int rows_block_local, int first_block, int num_blocks,
                              void* stream);

/*
 * One decode step of one attention layer in a single call (paper Fig. 3): the compressed-K
 * update for the block that has just filled (Sec. 3.2, skipped when k_nope is NULL), gate scoring
 * and token-budget selection (Eq. 1a/1c, Sec. 3.1), block-sparse decode over the selected
 * blocks (Sec. 3.3).  The results are those of the three calls
 *     seer_kcomp_append(.., first_block = -1) ; seer_gate_select(.., scores_in = NULL) ; seer_sparse_decode
 * on `stream`, with one host round trip instead of three.  (The launches go out as gate, attention,
 * append: the block that has just filled is the sequence's last block, which the gate takes without
 * scoring it, so the entry the append writes is first read in the next step.  When gate->max_blocks
 * blocks cover kv->max_seq_len, the attention kernel knows every list's length from the sequence
 * lengths and the budget; the gate kernel then marks each list as it finishes it and the attention
 * kernel starts on a sequence's blocks as soon as that list is marked, with a bounded wait that ends
 * in SEER_ERR_TIMEOUT.  SEER_STEP_LIST_FLAGS=0 in the environment at seer_create makes it wait for
 * the whole gate kernel instead; the results are the same.)
 *  block_idx / block_cnt / max_sel: caller-owned scratch for the selected lists (they are
 *  outputs too: the lists the attention used).  Other arguments as in the three calls;
 *  kv->seq_lens is used as the sequence lengths of all three.
 */
seer_status seer_decode_step(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv, const seer_gate* gate,
                             const void* q, const void* q_nope, const void* k_nope,
                             int64_t k_nope_stride_batch, int64_t k_nope_stride_head, int64_t k_nope_stride_token,
                             int k_nope_rows_block_local, int token_budget,
                             int32_t* block_idx, int32_t* block_cnt, int max_sel,
                             void* out, float* lse, void* stream);

/*
 * The same step for q_len query tokens per sequence (1 <= q_len <= 8; the sequences have just grown
 * by q_len tokens): seer_kcomp_append(.., first_block = -q_len) ; seer_gate_select_multi ;
 * seer_sparse_decode_multi, on `stream`.  q, q_nope: [B,q_len,Hq,d]; out: [B,q_len,Hq,d];
 * lse: [B,q_len,Hq] or NULL.  Other arguments as in seer_decode_step.
 */
seer_status seer_decode_step_multi(seer_ctx* ctx, const seer_shape* shape, const seer_kv* kv, const seer_gate* gate,
                                   const void* q, const void* q_nope, int q_len, const void* k_nope,
                                   int64_t k_nope_stride_batch, int64_t k_nope_stride_head,
                                   int64_t k_nope_stride_token, int k_nope_rows_block_local, int token_budget,
                                   int32_t* block_idx, int32_t* block_cnt, int max_sel, void* out, float* lse,
                                   void* stream);

/*
 * seer_gate_select without a context and without any allocation.  (The paper has no counterpart:
 * this entry point exists for hosts of the library, not for the method.)
 *
 * Some callers may not allocate device memory at all: an inference server that hands every byte
 * of HBM to its own pool at start-up and forbids cudaMalloc afterwards (a late allocation can
 * fail, or stall the GPU, under its memory plan), or code that runs inside a region where the
 * CUDA allocator must not be entered.  seer_create allocates a workspace, so those callers
 * cannot have a context.  This call computes exactly what seer_gate_select computes from
 * q_nope (same kernels, same results) but keeps the scratch it needs -- per-unit tickets, the gate
 * query, and the block scores unless scores_out is given -- in an array of
 * SEER_STATIC_SCRATCH_BYTES that is part of the library image.  Every GPU on which the library
 * is used holds one copy of that array from first use until the process exits.
 *
 *  - It calls no cudaMalloc / cudaFree and no allocating library routine.
 *  - Up to 8192 compressed keys per unit (max_blocks <= 8192) the gate is one kernel that keeps its
 *    intermediate results in shared memory; the array is then not needed and any B*Hkv is accepted.
 *    Beyond that the gate runs as two kernels that pass the gate query and the scores through the
 *    array.  Such a call needs 256 + 4*B*Hkv + 4*B*Hkv*d_gate (+ 4*B*Hkv*max_blocks without
 *    scores_out) bytes, each part rounded up to 256; if that exceeds the array the call returns
 *    SEER_ERR_WORKSPACE and launches nothing, and `err` says how much was needed.  (Example that
 *    fits: B*Hkv = 16, d_gate 128, max_blocks 16000.)
 *  - The first call on a device looks up the array's device address (cudaGetSymbolAddress, with
 *    that device made current).  Make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps the previous call's contents.  The
 *    call clears the part that must start at zero (the tickets) on `stream`; two calls that
 *    overlap on the GPU (different streams without ordering, or concurrent host threads) race on
 *    it and give wrong results.  Order them.
 *  - err / err_len: optional caller buffer that receives a one-line message on failure.
 * Arguments otherwise as for seer_gate_select (scores_in is not offered: selection on given
 * scores needs no scratch and no context-free variant).
 */
#define SEER_STATIC_SCRATCH_BYTES (1 << 20)
seer_status seer_gate_select_static(int device, const seer_shape* shape, const seer_gate* gate,
                                    const int32_t* seq_lens, const void* q_nope, int token_budget,
                                    int32_t* block_idx, int32_t* block_cnt, int max_sel,
                                    float* scores_out, void* stream, char* err, size_t err_len);

#ifdef __cplusplus
}
#endif
#endif /* SEER_H_ */
