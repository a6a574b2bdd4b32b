/*
 * dsa_oracle.c -- float64 CPU oracle for diagonal-aware sparse decode attention.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is the slow, plain statement of what the
 * CUDA library must compute.  Only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may load it; the product path never does.  It shares no code, header, table or helper
 * with the CUDA sources.
 *
 * What it follows (paper = "Understanding and Exploiting Diagonal Attention Sparsity in
 * Autoregressive Image Generation"):
 *   - dsa_oracle_replay        : Algorithm 1 taken literally, step by step, in the paper's
 *                                notation (window, skip_idx, idx, the three phases), with the
 *                                selection rule of its phase 2 pluggable (see below).
 *   - dsa_oracle_attend        : Attn(Q_t, K_p + K[idx], V_p + V[idx]) of Algorithm 1 -- plain
 *                                softmax attention of one query over the concatenation of the
 *                                prompt keys and the kept decode keys, written as its definition.
 *   - dsa_oracle_decode        : the loop over requests and heads around those two.
 *   - dsa_oracle_combine       : merge of partial softmax results by log-sum-exp.  The paper has
 *                                no such step; it is the exact identity
 *                                softmax over A u B = weighted mix of softmax over A and over B.
 *   - dsa_oracle_select_argmin : phase-2 selection of Algorithm 1 (softmax over the decode idx
 *                                only, argmin), for one step.
 *
 * Readings of the paper taken here (each is also listed in the design notes of the repository):
 *   R1  The window of Algorithm 1 is written [max(0,t-N_r) .. t], which has N_r+1 entries once
 *       t >= N_r; phase 3 evicts K[t-N_r] in the same step, so N_r entries stay.  The paper's
 *       example (N_r = 7, N_att = 4, three skips, four keys attended from then on) fixes this.
 *   R2  Phase 1 is t < N_att-1 (the algorithm), not t < N_att (one sentence of the prose); the
 *       example selects first at t = 3 with N_att = 4.
 *   R3  An entry appended to skip_idx at step s is not skipped at step s (Section 4, item 2).
 *   R4  Selection by "grid locality" (selector 1) is not in the paper: it stands in for the
 *       data-dependent argmin when no trained model is at hand.  With stride = tokens per image
 *       row, the column distance of a key that lies o tokens behind the query is
 *       d(o) = min(o mod stride, stride - o mod stride); at every selection step the attended
 *       key with the LARGEST (d(o), o) is appended to skip_idx.        [parity unpinned by the paper]
 *   R5  Argmin ties go to the lowest cache index.                       [parity unpinned by the paper]
 *   R6  Attn uses logits sm_scale * q.k, softmax jointly over prompt and kept decode keys;
 *       lse is the natural-log log-sum-exp of those logits.
 *   R8  Sink variants (Section 5.1, "Diagonal + sink4", StreamingLLM): the first n_sink decode
 *       tokens are attended at every step on top of what Algorithm 1 attends; the selection runs
 *       unchanged with its own N_att (callers pass N_att = budget - n_sink), except that a sink
 *       is never a candidate of the argmin (Section 5.1: the selection fills the other slots only).
 *                                                                        [parity unpinned]
 *   R7  A request with no decode token yet (seq_len == prompt_len) attends its prompt only; a
 *       request with seq_len == 0 yields out = 0 and lse = -inf.
 *
 * Pins: tests/test_oracle_pins.py (the paper's worked example, closed forms, brute force,
 * special cases that reduce to textbook attention).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORA_OK 0
#define ORA_BAD_ARG (-1)
#define ORA_BAD_TRACE (-2)
#define ORA_NO_MEM (-3)

enum { ORA_F64 = 0, ORA_F32 = 1, ORA_BF16 = 2 };
enum { ORA_SEL_TRACE = 0, ORA_SEL_GRID = 1, ORA_SEL_ARGMIN = 2 };
enum { ORA_MODE_DENSE = 0, ORA_MODE_WINDOW = 1, ORA_MODE_GRID = 2, ORA_MODE_LIST = 3 };

static double load_elem(const void *base, int dtype, int64_t i)
{
    if (dtype == ORA_F64) return ((const double *)base)[i];
    if (dtype == ORA_F32) return (double)((const float *)base)[i];
    /* bfloat16 bit pattern: the upper half of an IEEE float32 */
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[i]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

int dsa_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int dsa_oracle_select_argmin(const void *q_row, const void *k_base, int dtype,
                             const int64_t *k_rows, int32_t n_idx, int32_t D, double sm_scale,
                             int32_t *j_star, double *w_out);

/* what the argmin selector needs: the query of every step and the decode keys */
typedef struct {
    const void *q_steps;      /* query of step t starts at element t * q_step_stride */
    int64_t q_step_stride;
    const void *k_base;
    const int64_t *k_rows;    /* element offset of decode key j */
    int dtype;
    int32_t D;
    double sm_scale;
    int32_t n_sink;           /* decode keys 0 .. n_sink-1 are sinks: never candidates (R8) */
} argmin_ctx;

/* column distance on the raster grid of a key o tokens behind the query (reading R4) */
static int grid_col_dist(int o, int stride)
{
    int r = o % stride;
    return r < stride - r ? r : stride - r;
}

/*
 * Algorithm 1, literally.  Runs decode steps 0 .. t_final and returns what step t_final attends.
 *
 *   selector ORA_SEL_TRACE : the k-th selection (k = 0,1,..) appends the key that lies trace[k]
 *                            tokens behind the query of that step, i.e. idx entry s - trace[k];
 *                            the trace records the outcome of the paper's argmin so that the
 *                            attention path can be checked without re-deciding near-ties.
 *   selector ORA_SEL_GRID  : reading R4.
 *
 *   idx_out   [>= N_r]     : decode-relative key indices attended at step t_final, ascending
 *   skip_out  [>= N_r]     : skip_idx as it stands at the END of step t_final (after an append)
 * Returns ORA_OK, ORA_BAD_ARG, ORA_BAD_TRACE (trace too short, or names a key not in idx).
 */
static int replay_core(int32_t t_final, int32_t N_r, int32_t N_att, int32_t selector,
                       const int32_t *trace, int32_t trace_len, int32_t stride, const argmin_ctx *ctx,
                       int32_t *idx_out, int32_t *n_idx_out,
                       int32_t *skip_out, int32_t *n_skip_out,
                       int32_t *trace_out, int32_t *n_trace_out)
{
    if (t_final < 0 || N_att < 1 || N_r < N_att) return ORA_BAD_ARG;
    if (selector == ORA_SEL_GRID && stride < 1) return ORA_BAD_ARG;
    if (selector != ORA_SEL_GRID && selector != ORA_SEL_TRACE && selector != ORA_SEL_ARGMIN) return ORA_BAD_ARG;
    if (selector == ORA_SEL_ARGMIN && (!ctx || ctx->n_sink >= N_att)) return ORA_BAD_ARG;

    int32_t *skip_idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)(N_r + 1));
    int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)(N_r + 1));
    /* present[j]: K[j] has not been evicted; in_skip[j]: j is currently in skip_idx */
    unsigned char *present = (unsigned char *)malloc((size_t)t_final + 2);
    unsigned char *in_skip = (unsigned char *)calloc((size_t)t_final + 2, 1);
    if (!skip_idx || !idx || !present || !in_skip) {
        free(skip_idx); free(idx); free(present); free(in_skip);
        return ORA_NO_MEM;
    }
    memset(present, 1, (size_t)t_final + 2);
    int n_skip = 0, n_idx = 0, n_sel = 0, rc = ORA_OK;

    for (int32_t t = 0; t <= t_final && rc == ORA_OK; ++t) {
        int32_t w_lo = t - N_r > 0 ? t - N_r : 0;        /* window <- [max(0,t-N_r) .. t] */
        if (t < N_att - 1) {
            /* Phase 1: full attention, idx <- window */
            n_idx = 0;
            for (int32_t j = w_lo; j <= t; ++j) if (present[j]) idx[n_idx++] = j;
        } else {
            if (t >= N_r) {
                /* Phase 3: evict the oldest key, K[t-N_r] <- empty */
                present[t - N_r] = 0;
            }
            /* Phases 2 and 3: skip_idx <- [j+1 for j in skip_idx] */
            for (int i = 0; i < n_skip; ++i) in_skip[skip_idx[i]] = 0;
            for (int i = 0; i < n_skip; ++i) { skip_idx[i] += 1; in_skip[skip_idx[i]] = 1; }
            /* idx <- window - skip_idx */
            n_idx = 0;
            for (int32_t j = w_lo; j <= t; ++j)
                if (present[j] && !in_skip[j]) idx[n_idx++] = j;
            /* (attention over K_p + K[idx] happens here) */
            if (t < N_r && n_skip < N_r - N_att) {
                /* Phase 2 only: select the newly skipped key among idx */
                int32_t chosen = -1;
                if (selector == ORA_SEL_TRACE) {
                    if (n_sel >= trace_len) { rc = ORA_BAD_TRACE; break; }
                    int32_t want = t - trace[n_sel];
                    for (int i = 0; i < n_idx; ++i) if (idx[i] == want) chosen = want;
                    if (chosen < 0) { rc = ORA_BAD_TRACE; break; }
                } else if (selector == ORA_SEL_ARGMIN) {
                    /* w <- softmax(Q_t . K[idx]^T); j* <- argmin_j w[j]   (sinks are not in the race) */
                    int64_t *rows = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n_idx + 1));
                    int32_t *cand = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_idx + 1));
                    if (!rows || !cand) { free(rows); free(cand); rc = ORA_NO_MEM; break; }
                    int n_cand = 0;
                    for (int i = 0; i < n_idx; ++i)
                        if (idx[i] >= ctx->n_sink) { cand[n_cand] = idx[i]; rows[n_cand++] = ctx->k_rows[idx[i]]; }
                    int32_t j_star = -1;
                    size_t esz = ctx->dtype == ORA_F64 ? 8 : (ctx->dtype == ORA_F32 ? 4 : 2);
                    const void *q_t = (const char *)ctx->q_steps + (size_t)t * (size_t)ctx->q_step_stride * esz;
                    rc = dsa_oracle_select_argmin(q_t, ctx->k_base, ctx->dtype, rows, n_cand, ctx->D,
                                                  ctx->sm_scale, &j_star, NULL);
                    if (rc == ORA_OK) chosen = cand[j_star];
                    free(rows); free(cand);
                    if (rc != ORA_OK) break;
                } else {
                    int best_d = -1, best_o = -1;
                    for (int i = 0; i < n_idx; ++i) {
                        int o = t - idx[i];
                        int d = grid_col_dist(o, stride);
                        if (d > best_d || (d == best_d && o > best_o)) {
                            best_d = d; best_o = o; chosen = idx[i];
                        }
                    }
                }
                skip_idx[n_skip++] = chosen;              /* skip_idx.append(idx[j*]) */
                in_skip[chosen] = 1;
                if (trace_out) trace_out[n_sel] = t - chosen;   /* the same choice as a distance */
                ++n_sel;
            }
        }
    }
    if (rc == ORA_OK) {
        for (int i = 0; i < n_idx; ++i) idx_out[i] = idx[i];
        *n_idx_out = n_idx;
        if (skip_out) for (int i = 0; i < n_skip; ++i) skip_out[i] = skip_idx[i];
        if (n_skip_out) *n_skip_out = n_skip;
        if (n_trace_out) *n_trace_out = n_sel;
    }
    free(skip_idx); free(idx); free(present); free(in_skip);
    return rc;
}

int dsa_oracle_replay(int32_t t_final, int32_t N_r, int32_t N_att, int32_t selector,
                      const int32_t *trace, int32_t trace_len, int32_t stride,
                      int32_t *idx_out, int32_t *n_idx_out,
                      int32_t *skip_out, int32_t *n_skip_out)
{
    if (selector == ORA_SEL_ARGMIN) return ORA_BAD_ARG;
    return replay_core(t_final, N_r, N_att, selector, trace, trace_len, stride, NULL,
                       idx_out, n_idx_out, skip_out, n_skip_out, NULL, NULL);
}

/*
 * Algorithm 1 with its own selection rule (phase 2: softmax over the attended decode keys,
 * argmin), for one head of one sequence: runs steps 0 .. t_final with query q_steps[t] at step t
 * and decode key j at k_rows[j].  Returns what step t_final attends (idx_out, decode-relative)
 * and every selection made so far as distances behind the query of its step (trace_out, in
 * selection order) -- the form in which the attention calls take a trace.
 */
int dsa_oracle_replay_argmin(int32_t t_final, int32_t N_r, int32_t N_att, int32_t n_sink,
                             const void *q_steps, int64_t q_step_stride,
                             const void *k_base, int dtype, const int64_t *k_rows,
                             int32_t D, double sm_scale,
                             int32_t *idx_out, int32_t *n_idx_out,
                             int32_t *trace_out, int32_t *n_trace_out)
{
    argmin_ctx ctx = { q_steps, q_step_stride, k_base, k_rows, dtype, D, sm_scale, n_sink };
    return replay_core(t_final, N_r, N_att, ORA_SEL_ARGMIN, NULL, 0, 0, &ctx,
                       idx_out, n_idx_out, NULL, NULL, trace_out, n_trace_out);
}

/*
 * Phase-2 selection of Algorithm 1 for ONE step: w <- softmax(Q_t . K[idx]^T) over the decode
 * keys in idx only (no prompt keys), j* <- argmin_j w[j]; returns the position j* within idx.
 * Ties go to the lowest position (reading R5).  k_rows[i] is the element offset of key idx[i].
 */
int dsa_oracle_select_argmin(const void *q_row, const void *k_base, int dtype,
                             const int64_t *k_rows, int32_t n_idx, int32_t D, double sm_scale,
                             int32_t *j_star, double *w_out /* optional [n_idx] */)
{
    if (n_idx < 1 || D < 1) return ORA_BAD_ARG;
    double *s = (double *)malloc(sizeof(double) * (size_t)n_idx);
    if (!s) return ORA_NO_MEM;
    double mx = -INFINITY;
    for (int i = 0; i < n_idx; ++i) {
        double acc = 0.0;
        for (int d = 0; d < D; ++d)
            acc += load_elem(q_row, dtype, d) * load_elem(k_base, dtype, k_rows[i] + d);
        s[i] = acc * sm_scale;
        if (s[i] > mx) mx = s[i];
    }
    double sum = 0.0;
    for (int i = 0; i < n_idx; ++i) { s[i] = exp(s[i] - mx); sum += s[i]; }
    int best = 0;
    for (int i = 0; i < n_idx; ++i) {
        s[i] /= sum;
        if (s[i] < s[best]) best = i;
    }
    if (w_out) for (int i = 0; i < n_idx; ++i) w_out[i] = s[i];
    *j_star = best;
    free(s);
    return ORA_OK;
}

/*
 * Attn(q, K[rows], V[rows]): softmax attention of one query over n_rows key/value rows.
 *   s_j = sm_scale * sum_d q[d] k_j[d];  lse = ln sum_j e^{s_j};  out = sum_j e^{s_j - lse} v_j
 * k_rows[j] / v_rows[j] are element offsets of row j from k_base / v_base.
 */
int dsa_oracle_attend(const void *q_row, const void *k_base, const void *v_base, int dtype,
                      const int64_t *k_rows, const int64_t *v_rows, int32_t n_rows, int32_t D,
                      double sm_scale, double *out /* [D] */, double *lse)
{
    if (D < 1 || n_rows < 0) return ORA_BAD_ARG;
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    if (n_rows == 0) { *lse = -INFINITY; return ORA_OK; }
    double *s = (double *)malloc(sizeof(double) * (size_t)n_rows);
    if (!s) return ORA_NO_MEM;
    double mx = -INFINITY;
    for (int j = 0; j < n_rows; ++j) {
        double acc = 0.0;
        for (int d = 0; d < D; ++d)
            acc += load_elem(q_row, dtype, d) * load_elem(k_base, dtype, k_rows[j] + d);
        s[j] = acc * sm_scale;
        if (s[j] > mx) mx = s[j];
    }
    double sum = 0.0;
    for (int j = 0; j < n_rows; ++j) sum += exp(s[j] - mx);
    double l = mx + log(sum);
    for (int j = 0; j < n_rows; ++j) {
        double w = exp(s[j] - l);
        for (int d = 0; d < D; ++d) out[d] += w * load_elem(v_base, dtype, v_rows[j] + d);
    }
    *lse = l;
    free(s);
    return ORA_OK;
}

/*
 * Merge n_split partial results of one query: lse = ln sum_i e^{lse_i},
 * out = sum_i e^{lse_i - lse} out_i.  A part with lse_i = -inf holds nothing and is ignored.
 * Layouts: out_part [rows, n_split, D], lse_part [rows, n_split], out [rows, D], lse [rows].
 */
int dsa_oracle_combine(const double *out_part, const double *lse_part, int64_t rows,
                       int32_t n_split, int32_t D, double *out, double *lse)
{
    if (rows < 0 || n_split < 1 || D < 1) return ORA_BAD_ARG;
    for (int64_t r = 0; r < rows; ++r) {
        const double *lp = lse_part + r * n_split;
        double mx = -INFINITY;
        for (int i = 0; i < n_split; ++i) if (lp[i] > mx) mx = lp[i];
        for (int d = 0; d < D; ++d) out[r * D + d] = 0.0;
        if (mx == -INFINITY) { lse[r] = -INFINITY; continue; }
        double sum = 0.0;
        for (int i = 0; i < n_split; ++i) if (lp[i] != -INFINITY) sum += exp(lp[i] - mx);
        double l = mx + log(sum);
        for (int i = 0; i < n_split; ++i) {
            if (lp[i] == -INFINITY) continue;
            double w = exp(lp[i] - l);
            for (int d = 0; d < D; ++d)
                out[r * D + d] += w * out_part[(r * n_split + i) * D + d];
        }
        lse[r] = l;
    }
    return ORA_OK;
}

/*
 * Kept cache rows of one (request, mask head): the whole prompt [0, L_p) followed by the decode
 * keys Algorithm 1 attends at step t = p - 1, as cache positions L_p + j, ascending.
 *   mode DENSE  : every cached token [0, L_p + p)
 *   mode WINDOW : Algorithm 1 with nothing to skip (N_att = N_r): prompt + the N_r latest tokens
 *   mode GRID   : Algorithm 1, selector ORA_SEL_GRID
 *   mode LIST   : Algorithm 1, selector ORA_SEL_TRACE with the given trace
 * plus the first n_sink decode tokens (R8).
 * kept_out needs room for L_p + min(p, N_r + n_sink) entries (L_p + p for DENSE).
 */
int dsa_oracle_kept(int32_t mode, int32_t L_p, int32_t p, int32_t N_r, int32_t N_att,
                    int32_t stride, const int32_t *trace, int32_t trace_len, int32_t n_sink,
                    int32_t *kept_out, int32_t *n_kept_out)
{
    if (L_p < 0 || p < 0 || n_sink < 0) return ORA_BAD_ARG;
    int n = 0;
    for (int j = 0; j < L_p; ++j) kept_out[n++] = j;          /* K_p: always attended in full */
    if (p == 0) { *n_kept_out = n; return ORA_OK; }            /* reading R7 */
    if (mode == ORA_MODE_DENSE) {
        for (int j = 0; j < p; ++j) kept_out[n++] = L_p + j;
        *n_kept_out = n;
        return ORA_OK;
    }
    int32_t n_idx = 0, rc;
    int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)(N_r + 1));
    if (!idx) return ORA_NO_MEM;
    if (mode == ORA_MODE_WINDOW)
        rc = dsa_oracle_replay(p - 1, N_r, N_r, ORA_SEL_TRACE, NULL, 0, 0, idx, &n_idx, NULL, NULL);
    else if (mode == ORA_MODE_GRID)
        rc = dsa_oracle_replay(p - 1, N_r, N_att, ORA_SEL_GRID, NULL, 0, stride, idx, &n_idx, NULL, NULL);
    else if (mode == ORA_MODE_LIST)
        rc = dsa_oracle_replay(p - 1, N_r, N_att, ORA_SEL_TRACE, trace, trace_len, 0, idx, &n_idx, NULL, NULL);
    else
        rc = ORA_BAD_ARG;
    if (rc == ORA_OK) {
        /* sinks: decode tokens 0 .. n_sink-1, attended whether or not idx holds them (R8) */
        int i = 0;
        for (int j = 0; j < n_sink && j < p; ++j) {
            while (i < n_idx && idx[i] < j) kept_out[n++] = L_p + idx[i++];
            if (i < n_idx && idx[i] == j) ++i;
            kept_out[n++] = L_p + j;
        }
        while (i < n_idx) kept_out[n++] = L_p + idx[i++];
        *n_kept_out = n;
    }
    free(idx);
    return rc;
}

/*
 * One decode-attention call over a batch: for every request b and query head h, the kept rows of
 * its mask head, then dsa_oracle_attend on them.  Query head h reads kv head h / (H_q / H_kv).
 *
 * Cache layout (element strides, the last dimension D is contiguous):
 *   block_table == NULL : token s of request b, kv head g at  b*stride_b + s*stride_tok + g*stride_head
 *   block_table != NULL : token s lives in block block_table[b*max_blocks + s/block_size] at
 *                         block*stride_b + (s % block_size)*stride_tok + g*stride_head
 * q [B, H_q, D] contiguous.  seq_len[b] = L_p + p, prompt_len[b] = L_p.
 * trace: [B, mask_heads, trace_len] for mode LIST; mask_heads in {1, H_kv, H_q}; mask head of
 * query head h is 0, h / G or h respectively.
 * kept_idx_out (optional) [B, mask_heads, max_kept], kept_cnt_out [B, mask_heads].
 * out [B, H_q, D] and lse [B, H_q] in float64.
 */
int dsa_oracle_decode(int32_t B, int32_t H_q, int32_t H_kv, int32_t D, int32_t dtype,
                      const void *q, const void *k_cache, const void *v_cache,
                      int64_t stride_b, int64_t stride_tok, int64_t stride_head,
                      const int32_t *seq_len, const int32_t *prompt_len,
                      const int32_t *block_table, int32_t max_blocks, int32_t block_size,
                      int32_t mode, int32_t N_r, int32_t N_att, int32_t stride_grid,
                      const int32_t *trace, int32_t mask_heads, int32_t trace_len, int32_t n_sink,
                      double sm_scale, double *out, double *lse,
                      int32_t *kept_idx_out, int32_t *kept_cnt_out, int32_t max_kept,
                      int32_t n_threads)
{
    if (B < 0 || H_q < 1 || H_kv < 1 || H_q % H_kv || D < 1) return ORA_BAD_ARG;
    if (mask_heads != 1 && mask_heads != H_kv && mask_heads != H_q) return ORA_BAD_ARG;
    if (block_table && (block_size < 1 || max_blocks < 1)) return ORA_BAD_ARG;
    const int G = H_q / H_kv;
    int status = ORA_OK;
    (void)n_threads;
#ifdef _OPENMP
    if (n_threads < 1) n_threads = omp_get_max_threads();
#pragma omp parallel for collapse(2) schedule(dynamic, 1) num_threads(n_threads)
#endif
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < H_q; ++h) {
            int32_t S = seq_len[b], L_p = prompt_len[b];
            if (S < 0) S = 0;
            if (L_p > S) L_p = S;
            if (L_p < 0) L_p = 0;
            int32_t p = S - L_p;
            int mh = mask_heads == 1 ? 0 : (mask_heads == H_kv ? h / G : h);
            int g = h / G;
            int32_t cap = S + 1, n_kept = 0;
            int32_t *kept = (int32_t *)malloc(sizeof(int32_t) * (size_t)cap);
            int64_t *rows = (int64_t *)malloc(sizeof(int64_t) * (size_t)cap);
            int rc = (kept && rows) ? ORA_OK : ORA_NO_MEM;
            if (rc == ORA_OK) {
                const int32_t *tr = (mode == ORA_MODE_LIST && trace)
                    ? trace + ((int64_t)b * mask_heads + mh) * trace_len : NULL;
                rc = dsa_oracle_kept(mode, L_p, p, N_r, N_att, stride_grid, tr, trace_len, n_sink, kept, &n_kept);
            }
            if (rc == ORA_OK) {
                for (int i = 0; i < n_kept; ++i) {
                    int32_t s = kept[i];
                    if (block_table) {
                        int64_t blk = block_table[(int64_t)b * max_blocks + s / block_size];
                        rows[i] = blk * stride_b + (int64_t)(s % block_size) * stride_tok + g * stride_head;
                    } else {
                        rows[i] = (int64_t)b * stride_b + (int64_t)s * stride_tok + g * stride_head;
                    }
                }
                const char *qb = (const char *)q;
                size_t esz = dtype == ORA_F64 ? 8 : (dtype == ORA_F32 ? 4 : 2);
                const void *q_row = qb + ((size_t)b * H_q + h) * (size_t)D * esz;
                rc = dsa_oracle_attend(q_row, k_cache, v_cache, dtype, rows, rows, n_kept, D, sm_scale,
                                       out + ((int64_t)b * H_q + h) * D, lse + (int64_t)b * H_q + h);
                /* one writer per (request, mask head): the first query head that maps to it */
                int first_h = mask_heads == H_q ? h : (mask_heads == H_kv ? g * G : 0);
                if (rc == ORA_OK && kept_cnt_out && h == first_h) {
                    kept_cnt_out[(int64_t)b * mask_heads + mh] = n_kept;
                    if (kept_idx_out)
                        for (int i = 0; i < n_kept && i < max_kept; ++i)
                            kept_idx_out[((int64_t)b * mask_heads + mh) * max_kept + i] = kept[i];
                }
            }
            free(kept); free(rows);
            if (rc != ORA_OK) {
#ifdef _OPENMP
#pragma omp critical
#endif
                status = rc;
            }
        }
    }
    return status;
}
