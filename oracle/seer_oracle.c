/*
 * seer_oracle.c -- plain fp64 CPU oracle for the SeerAttention-R decode path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file defines what the GPU library must
 * compute; it is slow on purpose (direct definitions, two-pass softmax, full
 * sorts) and is never part of the product path.  It shares no source, header,
 * table or helper with the CUDA code.  Only the test-suite, the smoke check and
 * the benchmark's CPU-baseline leg may load it.
 *
 * Every bf16 input is widened exactly to double; all arithmetic is double.
 * Parallelism: an OpenMP "parallel for" over independent (sequence, head)
 * units, nothing else (no blocking, no fusion, no reordering of the sums).
 *
 * Conventions shared by all functions
 *   B  batch, Hq query heads, Hkv KV heads, g = Hq/Hkv, d head dim,
 *   b  block size, L_i KV length of sequence i (includes the current token),
 *   n_i = ceil(L_i / b) blocks.  Query head hq belongs to KV head hq / g
 *   (contiguous groups; the grouping the paper describes for GQA sharing,
 *   Sec. 2.2 "Aggregation of Query Heads").
 *   K/V/K_nope are addressed as base[i*sb + h*sh + t*st + c] (element
 *   strides, channel stride 1).
 *
 * Pins (tests marked "not gpu"): closed forms of softmax attention, dense ==
 * 100% selection, an independent streaming/LSE-merge formulation in numpy,
 * torch's fp64 attention, shift and permutation invariances (attention);
 * constant-block / identity-weight / position-0 cases, a complex-number
 * restatement of the rotation, norm and relative-position invariants (gate);
 * brute-force lexicographic sort with crafted ties (selection).
 * Parity unpinned: the rotary convention itself (pairing c <-> c + d_gate/2,
 * base theta) against the authors' trained gates -- the paper only says that
 * RoPE is re-applied inside the gate (Sec. 2.2 "Positional Embedding").
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef uint16_t bf16_t;

static double bf16_to_f64(bf16_t u)
{
    uint32_t w = ((uint32_t)u) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* Round a double to the nearest bf16 (ties to even) in one rounding step. */
static bf16_t f64_to_bf16(double x)
{
    if (isnan(x)) return 0x7fc0;
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7f80;
    int e;
    (void)frexp(a, &e);           /* a = m * 2^e, m in [0.5, 1) */
    int ex = e - 1;               /* a in [2^ex, 2^(ex+1)) */
    if (ex < -126) ex = -126;     /* subnormal quantum */
    double quantum = ldexp(1.0, ex - 7);
    double r = nearbyint(a / quantum) * quantum;   /* default mode: ties to even */
    if (r >= ldexp(1.0, 128)) return sign | 0x7f80;
    float f = (float)r;           /* exact: r has at most 8 significant bits */
    uint32_t w;
    memcpy(&w, &f, sizeof w);
    return sign | (uint16_t)(w >> 16);
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Exposed so that tests can pin the rounding helper itself. */
uint16_t oracle_round_bf16(double x) { return f64_to_bf16(x); }

/* ------------------------------------------------------------------------- */
/* Attention of one query head over an explicit token mask.                  */
/* o = sum_t softmax_t(scale <q,k_t>) v_t ,  lse = log sum_t exp(scale <q,k_t>)
 * over the tokens with use[t] != 0 (use == NULL: all t < L).  Two passes:
 * scores and their maximum first, then the normalised weighted sum.         */
static void attend_one(const bf16_t *q, const bf16_t *k, const bf16_t *v,
                       int64_t st, int L, int d, double scale,
                       const unsigned char *use, double *o, double *lse)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
    double mx = -INFINITY;
    int any = 0;
    for (int t = 0; t < L; ++t) {
        if (use && !use[t]) continue;
        double acc = 0.0;
        for (int c = 0; c < d; ++c)
            acc += bf16_to_f64(q[c]) * bf16_to_f64(k[(int64_t)t * st + c]);
        s[t] = acc * scale;
        if (s[t] > mx) mx = s[t];
        any = 1;
    }
    for (int c = 0; c < d; ++c) o[c] = 0.0;
    if (!any) {                       /* empty selection: o = 0, lse = -inf */
        *lse = -INFINITY;
        free(s);
        return;
    }
    double z = 0.0;
    for (int t = 0; t < L; ++t) {
        if (use && !use[t]) continue;
        z += exp(s[t] - mx);
    }
    for (int t = 0; t < L; ++t) {
        if (use && !use[t]) continue;
        double p = exp(s[t] - mx) / z;
        for (int c = 0; c < d; ++c)
            o[c] += p * bf16_to_f64(v[(int64_t)t * st + c]);
    }
    *lse = mx + log(z);
    free(s);
}

/* Dense softmax attention for decoding: the textbook definition over every
 * cached token t < L_i (the baseline the paper's kernel is compared with,
 * Sec. 4.4).  q, out: [B,Hq,d]; lse: [B,Hq]. */
void oracle_dense(const bf16_t *q, const bf16_t *k, const bf16_t *v,
                  int64_t sb, int64_t sh, int64_t st,
                  const int32_t *seq_lens, int B, int Hq, int Hkv, int d,
                  double scale, double *out, double *lse)
{
    int g = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int i = 0; i < B; ++i)
        for (int hq = 0; hq < Hq; ++hq) {
            int h = hq / g;
            attend_one(q + ((int64_t)i * Hq + hq) * d,
                       k + i * sb + h * sh, v + i * sb + h * sh, st,
                       seq_lens[i], d, scale, NULL,
                       out + ((int64_t)i * Hq + hq) * d,
                       lse + (int64_t)i * Hq + hq);
        }
}

/* Block-sparse attention (Sec. 3.3): the same sum restricted to the tokens of
 * the blocks listed for (sequence, KV head): t in [j*b, min((j+1)*b, L_i)) for
 * j in the list.  Negative, out-of-range and repeated entries are ignored.
 * block_idx: [B,Hkv,max_sel]; block_cnt: [B,Hkv] or NULL (= read all max_sel
 * entries).  All query heads of a group use the list of their KV head. */
void oracle_sparse(const bf16_t *q, const bf16_t *k, const bf16_t *v,
                   int64_t sb, int64_t sh, int64_t st,
                   const int32_t *seq_lens, const int32_t *block_idx,
                   const int32_t *block_cnt, int max_sel,
                   int B, int Hq, int Hkv, int d, int b,
                   double scale, double *out, double *lse)
{
    int g = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int i = 0; i < B; ++i)
        for (int hq = 0; hq < Hq; ++hq) {
            int h = hq / g;
            int L = seq_lens[i];
            int n = (L + b - 1) / b;
            unsigned char *use = (unsigned char *)calloc((size_t)(L > 0 ? L : 1), 1);
            int cnt = block_cnt ? block_cnt[i * Hkv + h] : max_sel;
            if (cnt > max_sel) cnt = max_sel;
            for (int e = 0; e < cnt; ++e) {
                int j = block_idx[((int64_t)i * Hkv + h) * max_sel + e];
                if (j < 0 || j >= n) continue;
                for (int t = j * b; t < (j + 1) * b && t < L; ++t) use[t] = 1;
            }
            attend_one(q + ((int64_t)i * Hq + hq) * d,
                       k + i * sb + h * sh, v + i * sb + h * sh, st,
                       L, d, scale, use,
                       out + ((int64_t)i * Hq + hq) * d,
                       lse + (int64_t)i * Hq + hq);
            free(use);
        }
}

/* Block-sparse attention for T query tokens per sequence (the query-level
 * parallelism of multi-token prediction / speculative decoding that Sec. 6
 * "Unify Sparse Prefill and Decoding" points to; the paper gives no formula, so
 * this is the causal definition written out).  The cache already holds all L_i
 * tokens, the last T of which are the queries' own: query t (0 <= t < T) sits at
 * position L_i - T + t and sees the cached tokens at positions <= its own, of
 * the blocks listed for its (sequence, KV head) -- one list for all T tokens,
 * as one list serves all heads of a group.  T = 1 is oracle_sparse.
 * q, out: [B,T,Hq,d]; lse: [B,T,Hq].  A query that sees no token gets a zero
 * row and lse = -inf.  Sequences with L_i < T: queries at negative positions
 * see nothing. */
void oracle_sparse_multi(const bf16_t *q, const bf16_t *k, const bf16_t *v,
                         int64_t sb, int64_t sh, int64_t st,
                         const int32_t *seq_lens, const int32_t *block_idx,
                         const int32_t *block_cnt, int max_sel,
                         int B, int T, int Hq, int Hkv, int d, int b,
                         double scale, double *out, double *lse)
{
    int g = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int i = 0; i < B; ++i)
        for (int hq = 0; hq < Hq; ++hq) {
            int h = hq / g;
            int L = seq_lens[i];
            int n = (L + b - 1) / b;
            unsigned char *listed = (unsigned char *)calloc((size_t)(L > 0 ? L : 1), 1);
            unsigned char *use = (unsigned char *)calloc((size_t)(L > 0 ? L : 1), 1);
            int cnt = block_cnt ? block_cnt[i * Hkv + h] : max_sel;
            if (cnt > max_sel) cnt = max_sel;
            for (int e = 0; e < cnt; ++e) {
                int j = block_idx[((int64_t)i * Hkv + h) * max_sel + e];
                if (j < 0 || j >= n) continue;
                for (int t = j * b; t < (j + 1) * b && t < L; ++t) listed[t] = 1;
            }
            for (int t = 0; t < T; ++t) {
                int pos = L - T + t;                      /* this query's own position */
                for (int x = 0; x < L; ++x) use[x] = (unsigned char)(listed[x] && x <= pos);
                int64_t row = ((int64_t)i * T + t) * Hq + hq;
                attend_one(q + row * d, k + i * sb + h * sh, v + i * sb + h * sh, st,
                           L, d, scale, use, out + row * d, lse + row);
            }
            free(use);
            free(listed);
        }
}

/* ------------------------------------------------------------------------- */
/* Rotary embedding inside the gate (Sec. 2.2 "Positional Embedding").  Reading
 * taken where the paper is silent: rotate-half pairing (c, c + dg/2), angle
 * pos * theta^(-2c/dg), applied over all dg channels. */
static void rope_f64(double *y, int dg, double pos, double theta)
{
    int half = dg / 2;
    for (int c = 0; c < half; ++c) {
        double ang = pos * pow(theta, -2.0 * (double)c / (double)dg);
        double cs = cos(ang), sn = sin(ang);
        double a = y[c], bb = y[c + half];
        y[c] = a * cs - bb * sn;
        y[c + half] = bb * cs + a * sn;
    }
}

/* Exposed for the invariants tests (norm, relative position). */
void oracle_rope(double *y, int dg, double pos, double theta) { rope_f64(y, dg, pos, theta); }

/* K branch of the gate (Eq. 1b; Sec. 2.2 "Pooling-based Compression of K"):
 * for block j of (sequence i, KV head h), per channel c the max, min and mean
 * over the block's b rows of K_nope (kernel = stride = b), concatenated as
 * [max | min | avg] (3d), multiplied by W_k[h] (dg x 3d), rotated at the
 * position of the block's first token (j*b), stored as bf16.
 * Blocks first_block .. first_block+num_blocks-1 of every sequence are
 * written; every one of them must be complete (all b rows present).
 * kc_bf16: [B,Hkv,max_blocks,dg]; kc_f64 (optional, same shape): unrounded. */
void oracle_kcomp(const bf16_t *k_nope, int64_t sb, int64_t sh, int64_t st,
                  const bf16_t *w_k, int B, int Hkv, int d, int dg, int b,
                  int first_block, int num_blocks, int max_blocks, double theta,
                  bf16_t *kc_bf16, double *kc_f64)
{
#pragma omp parallel for collapse(3) schedule(dynamic, 4)
    for (int i = 0; i < B; ++i)
        for (int h = 0; h < Hkv; ++h)
            for (int jj = 0; jj < num_blocks; ++jj) {
                int j = first_block + jj;
                if (j < 0 || j >= max_blocks) continue;
                double *feat = (double *)malloc(sizeof(double) * 3 * (size_t)d);
                double *y = (double *)malloc(sizeof(double) * (size_t)dg);
                const bf16_t *base = k_nope + i * sb + h * sh + (int64_t)j * b * st;
                for (int c = 0; c < d; ++c) {
                    double mx = -INFINITY, mn = INFINITY, sum = 0.0;
                    for (int t = 0; t < b; ++t) {
                        double x = bf16_to_f64(base[(int64_t)t * st + c]);
                        if (x > mx) mx = x;
                        if (x < mn) mn = x;
                        sum += x;
                    }
                    feat[c] = mx;
                    feat[d + c] = mn;
                    feat[2 * d + c] = sum / (double)b;
                }
                const bf16_t *w = w_k + (int64_t)h * dg * 3 * d;
                for (int r = 0; r < dg; ++r) {
                    double acc = 0.0;
                    for (int c = 0; c < 3 * d; ++c)
                        acc += bf16_to_f64(w[(int64_t)r * 3 * d + c]) * feat[c];
                    y[r] = acc;
                }
                rope_f64(y, dg, (double)j * (double)b, theta);
                int64_t o = (((int64_t)i * Hkv + h) * max_blocks + j) * dg;
                for (int r = 0; r < dg; ++r) {
                    kc_bf16[o + r] = f64_to_bf16(y[r]);
                    if (kc_f64) kc_f64[o + r] = y[r];
                }
                free(feat);
                free(y);
            }
}

/* Q branch of the gate and the block scores (Eq. 1a, 1c without the softmax,
 * which the token-budget method does not need, Sec. 3.1):
 *   x      = the g pre-RoPE query heads of KV head h laid end to end
 *            (index u*d + c for the u-th head of the group),
 *   q_gate = RoPE(W_q[h] x, position qpos[i]),
 *   score[j] = <q_gate, Kc[j]> / sqrt(dg)   for j < n_entries[i].
 * The query position is an explicit argument (the decode path passes L_i-1).
 * scores: [B,Hkv,max_blocks] (entries j >= n_entries[i] are left untouched);
 * q_gate_out (optional): [B,Hkv,dg]. */
void oracle_scores(const bf16_t *q_nope, const bf16_t *w_q, const bf16_t *kc,
                   const int32_t *n_entries, const int32_t *qpos,
                   int B, int Hq, int Hkv, int d, int dg, int max_blocks,
                   double theta, double *scores, double *q_gate_out)
{
    int g = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int i = 0; i < B; ++i)
        for (int h = 0; h < Hkv; ++h) {
            double *qg = (double *)malloc(sizeof(double) * (size_t)dg);
            const bf16_t *x = q_nope + ((int64_t)i * Hq + (int64_t)h * g) * d;
            const bf16_t *w = w_q + (int64_t)h * dg * g * d;
            for (int r = 0; r < dg; ++r) {
                double acc = 0.0;
                for (int c = 0; c < g * d; ++c)
                    acc += bf16_to_f64(w[(int64_t)r * g * d + c]) * bf16_to_f64(x[c]);
                qg[r] = acc;
            }
            rope_f64(qg, dg, (double)qpos[i], theta);
            if (q_gate_out)
                for (int r = 0; r < dg; ++r)
                    q_gate_out[((int64_t)i * Hkv + h) * dg + r] = qg[r];
            const bf16_t *kcb = kc + ((int64_t)i * Hkv + h) * max_blocks * dg;
            for (int j = 0; j < n_entries[i] && j < max_blocks; ++j) {
                double acc = 0.0;
                for (int r = 0; r < dg; ++r)
                    acc += qg[r] * bf16_to_f64(kcb[(int64_t)j * dg + r]);
                scores[((int64_t)i * Hkv + h) * max_blocks + j] = acc / sqrt((double)dg);
            }
            free(qg);
        }
}

/* ------------------------------------------------------------------------- */
/* Token-budget selection (Sec. 3.1) with the always-active last block
 * (Sec. 3.2, Fig. 3).  Readings taken where the paper is silent:
 *   k = min(max(1, budget / b), n_i)  (integer division),
 *   the last block n_i-1 is always in the list and counts against k,
 *   the other k-1 come from blocks [0, n_i-1) ranked by (score descending,
 *   index ascending); -0 and +0 compare equal; NaN ranks below every number;
 *   the list is emitted in ascending block order, padded with -1.
 * Scores are the fp32 values the selection is made on (compared as IEEE
 * floats, no arithmetic), so the result is exact.  scores: [B,Hkv,max_blocks];
 * block_idx: [B,Hkv,max_sel]; block_cnt: [B,Hkv]. */
typedef struct { float s; int32_t j; } cand_t;

static int cand_before(const void *pa, const void *pb)
{
    const cand_t *a = (const cand_t *)pa, *c = (const cand_t *)pb;
    int an = isnan(a->s), cn = isnan(c->s);
    if (an != cn) return an ? 1 : -1;            /* NaN after every number */
    if (!an) {
        if (a->s > c->s) return -1;
        if (a->s < c->s) return 1;
    }
    return (a->j > c->j) - (a->j < c->j);        /* equal scores: lower index first */
}

static int int_asc(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, c = *(const int32_t *)pb;
    return (a > c) - (a < c);
}

/* The `need` best of blocks [0, n-1) by (score descending, index ascending) plus the last block
 * n-1, ascending, -1 padded; returns the count. */
static int emit_best_and_last(const float *s, int n, int need, int max_sel, int32_t *dst)
{
    for (int e = 0; e < max_sel; ++e) dst[e] = -1;
    int ncand = n - 1;
    cand_t *cand = (cand_t *)malloc(sizeof(cand_t) * (size_t)(ncand > 0 ? ncand : 1));
    for (int j = 0; j < ncand; ++j) { cand[j].s = s[j]; cand[j].j = j; }
    qsort(cand, (size_t)ncand, sizeof(cand_t), cand_before);
    int m = 0;
    for (int e = 0; e < need && e < ncand; ++e) dst[m++] = cand[e].j;
    dst[m++] = n - 1;
    qsort(dst, (size_t)m, sizeof(int32_t), int_asc);
    free(cand);
    return m;
}

void oracle_select(const float *scores, const int32_t *seq_lens,
                   int B, int Hkv, int b, int max_blocks, int token_budget,
                   int max_sel, int32_t *block_idx, int32_t *block_cnt)
{
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int i = 0; i < B; ++i)
        for (int h = 0; h < Hkv; ++h) {
            int32_t *dst = block_idx + ((int64_t)i * Hkv + h) * max_sel;
            int L = seq_lens[i];
            int n = (L + b - 1) / b;
            if (n <= 0) {
                for (int e = 0; e < max_sel; ++e) dst[e] = -1;
                block_cnt[i * Hkv + h] = 0;
                continue;
            }
            int k = token_budget / b;
            if (k < 1) k = 1;
            if (k > n) k = n;
            if (k > max_sel) k = max_sel;
            const float *s = scores + ((int64_t)i * Hkv + h) * max_blocks;
            block_cnt[i * Hkv + h] = emit_best_and_last(s, n, k - 1, max_sel, dst);
        }
}

/* Threshold selection (Sec. 3.1, the second sparsify method): S = softmax of the gate scores
 * (Eq. 1c) over the blocks that have a compressed key, [0, n_i-1); the blocks with S_j > tau are
 * selected, and the last block always is (Sec. 3.2).  Readings where the paper is silent: the
 * last block takes no part in the normalisation (it has no valid entry); if more than
 * max_sel-1 blocks pass, the max_sel-1 highest-scoring are kept.  Scores must be finite.
 * probs_out (optional, [B,Hkv,max_blocks]): the softmax values, for tests. */
void oracle_select_threshold(const float *scores, const int32_t *seq_lens,
                             int B, int Hkv, int b, int max_blocks, double tau,
                             int max_sel, int32_t *block_idx, int32_t *block_cnt, double *probs_out)
{
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int i = 0; i < B; ++i)
        for (int h = 0; h < Hkv; ++h) {
            int32_t *dst = block_idx + ((int64_t)i * Hkv + h) * max_sel;
            int L = seq_lens[i];
            int n = (L + b - 1) / b;
            if (n <= 0) {
                for (int e = 0; e < max_sel; ++e) dst[e] = -1;
                block_cnt[i * Hkv + h] = 0;
                continue;
            }
            const float *s = scores + ((int64_t)i * Hkv + h) * max_blocks;
            int ncand = n - 1;
            double mx = -INFINITY, z = 0.0;
            for (int j = 0; j < ncand; ++j) if ((double)s[j] > mx) mx = (double)s[j];
            for (int j = 0; j < ncand; ++j) z += exp((double)s[j] - mx);
            int above = 0;
            for (int j = 0; j < ncand; ++j) {
                double pj = exp((double)s[j] - mx) / z;
                if (probs_out) probs_out[((int64_t)i * Hkv + h) * max_blocks + j] = pj;
                if (pj > tau) ++above;
            }
            int need = above;
            if (need > max_sel - 1) need = max_sel - 1;
            block_cnt[i * Hkv + h] = emit_best_and_last(s, n, need, max_sel, dst);
        }
}

/* ------------------------------------------------------------------------- */
/* The gate for T query tokens per sequence (the newest T cached tokens; see
 * oracle_sparse_multi).  The paper has no gate for several decode-time
 * queries; reading taken: every query token gets its own gate query, rotated
 * at its own position L_i - T + t; a block's score is the largest of the T
 * tokens' scores (a block that any token wants is wanted), over the blocks
 * that lie wholly before the first query token, j < j_f = floor((L_i - T)/b)
 * (all of them complete).  T = 1 is oracle_scores with n_entries = n_i - 1,
 * qpos = L_i - 1.  q_nope: [B,T,Hq,d]; scores: [B,Hkv,max_blocks], entries
 * j >= j_f untouched. */
void oracle_scores_multi(const bf16_t *q_nope, const bf16_t *w_q, const bf16_t *kc,
                         const int32_t *seq_lens, int T,
                         int B, int Hq, int Hkv, int d, int dg, int max_blocks, int b,
                         double theta, double *scores)
{
    int g = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int i = 0; i < B; ++i)
        for (int h = 0; h < Hkv; ++h) {
            int L = seq_lens[i];
            int jf = L - T > 0 ? (L - T) / b : 0;
            if (jf > max_blocks) jf = max_blocks;
            double *qg = (double *)malloc(sizeof(double) * (size_t)dg);
            double *best = scores + ((int64_t)i * Hkv + h) * max_blocks;
            const bf16_t *w = w_q + (int64_t)h * dg * g * d;
            const bf16_t *kcb = kc + ((int64_t)i * Hkv + h) * max_blocks * dg;
            for (int t = 0; t < T; ++t) {
                const bf16_t *x = q_nope + (((int64_t)i * T + t) * Hq + (int64_t)h * g) * d;
                for (int r = 0; r < dg; ++r) {
                    double acc = 0.0;
                    for (int c = 0; c < g * d; ++c)
                        acc += bf16_to_f64(w[(int64_t)r * g * d + c]) * bf16_to_f64(x[c]);
                    qg[r] = acc;
                }
                rope_f64(qg, dg, (double)(L - T + t), theta);
                for (int j = 0; j < jf; ++j) {
                    double acc = 0.0;
                    for (int r = 0; r < dg; ++r)
                        acc += qg[r] * bf16_to_f64(kcb[(int64_t)j * dg + r]);
                    acc /= sqrt((double)dg);
                    if (t == 0 || acc > best[j]) best[j] = acc;
                }
            }
            free(qg);
        }
}

/* Token-budget selection for T query tokens: the blocks that hold a query
 * token's own position, j_f .. n_i - 1 (one or two blocks for T <= b), are
 * always in the list and count against k = min(max(1, budget/b), n_i, max_sel);
 * the other k - (n_i - j_f) come from blocks [0, j_f) by (score descending,
 * index ascending).  If the forced blocks alone exceed max_sel the last max_sel
 * of them are kept.  T = 1 is oracle_select. */
void oracle_select_multi(const float *scores, const int32_t *seq_lens,
                         int B, int Hkv, int b, int max_blocks, int token_budget, int T,
                         int max_sel, int32_t *block_idx, int32_t *block_cnt)
{
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int i = 0; i < B; ++i)
        for (int h = 0; h < Hkv; ++h) {
            int32_t *dst = block_idx + ((int64_t)i * Hkv + h) * max_sel;
            for (int e = 0; e < max_sel; ++e) dst[e] = -1;
            int L = seq_lens[i];
            int n = (L + b - 1) / b;
            if (n <= 0) { block_cnt[i * Hkv + h] = 0; continue; }
            int jf = L - T > 0 ? (L - T) / b : 0;
            int k = token_budget / b;
            if (k < 1) k = 1;
            if (k > n) k = n;
            if (k > max_sel) k = max_sel;
            int forced = n - jf;
            if (forced > max_sel) forced = max_sel;
            int need = k - forced;
            if (need < 0) need = 0;
            if (need > jf) need = jf;
            if (need > max_blocks) need = max_blocks;
            const float *s = scores + ((int64_t)i * Hkv + h) * max_blocks;
            int ncand = jf < max_blocks ? jf : max_blocks;
            cand_t *cand = (cand_t *)malloc(sizeof(cand_t) * (size_t)(ncand > 0 ? ncand : 1));
            for (int j = 0; j < ncand; ++j) { cand[j].s = s[j]; cand[j].j = j; }
            qsort(cand, (size_t)ncand, sizeof(cand_t), cand_before);
            int m = 0;
            for (int e = 0; e < need && e < ncand; ++e) dst[m++] = cand[e].j;
            for (int j = n - forced; j < n; ++j) dst[m++] = j;
            qsort(dst, (size_t)m, sizeof(int32_t), int_asc);
            free(cand);
            block_cnt[i * Hkv + h] = m;
        }
}

/* Threshold selection for T query tokens per sequence (the reading taken for Sec. 3.1's second method
 * when several tokens are decoded at once; the paper has no such case): the per-block scores are the
 * maxima over the tokens (oracle_scores_multi); the softmax runs over the candidate blocks, those wholly
 * before the first query token, [0, jf) with jf = floor((L - T) / b); a candidate is selected if its
 * probability exceeds tau; the blocks that hold a query token, jf .. n-1, are always selected and take no
 * part in the normalisation; if more candidates pass than the list has room for beside the forced
 * blocks, the highest-scoring ones are kept (score descending, index ascending). */
void oracle_select_threshold_multi(const float *scores, const int32_t *seq_lens,
                                   int B, int Hkv, int b, int max_blocks, double tau, int T,
                                   int max_sel, int32_t *block_idx, int32_t *block_cnt, double *probs_out)
{
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int i = 0; i < B; ++i)
        for (int h = 0; h < Hkv; ++h) {
            int32_t *dst = block_idx + ((int64_t)i * Hkv + h) * max_sel;
            for (int e = 0; e < max_sel; ++e) dst[e] = -1;
            int L = seq_lens[i];
            int n = (L + b - 1) / b;
            if (n <= 0) { block_cnt[i * Hkv + h] = 0; continue; }
            int jf = L - T > 0 ? (L - T) / b : 0;
            int forced = n - jf;
            if (forced > max_sel) forced = max_sel;
            const float *s = scores + ((int64_t)i * Hkv + h) * max_blocks;
            int ncand = jf < max_blocks ? jf : max_blocks;
            double mx = -INFINITY, z = 0.0;
            for (int j = 0; j < ncand; ++j) if ((double)s[j] > mx) mx = (double)s[j];
            for (int j = 0; j < ncand; ++j) z += exp((double)s[j] - mx);
            int above = 0;
            for (int j = 0; j < ncand; ++j) {
                double pj = exp((double)s[j] - mx) / z;
                if (probs_out) probs_out[((int64_t)i * Hkv + h) * max_blocks + j] = pj;
                if (pj > tau) ++above;
            }
            int need = above;
            if (need > max_sel - forced) need = max_sel - forced;
            cand_t *cand = (cand_t *)malloc(sizeof(cand_t) * (size_t)(ncand > 0 ? ncand : 1));
            for (int j = 0; j < ncand; ++j) { cand[j].s = s[j]; cand[j].j = j; }
            qsort(cand, (size_t)ncand, sizeof(cand_t), cand_before);
            int m = 0;
            for (int e = 0; e < need && e < ncand; ++e) dst[m++] = cand[e].j;
            for (int j = n - forced; j < n; ++j) dst[m++] = j;
            qsort(dst, (size_t)m, sizeof(int32_t), int_asc);
            free(cand);
            block_cnt[i * Hkv + h] = m;
        }
}
