/*
 * fp64 CPU oracle for the verify-and-resample pass of speculative sampling.
 *
 * TEST INFRASTRUCTURE ONLY.  This file defines what the CUDA library must
 * compute; it shares no code with it and must never be linked into, imported
 * by, or called from the product path.  It is deliberately plain and slow:
 * one sequence after another, one position after another, two-pass softmax,
 * linear-scan inverse CDF, everything in double precision, sums taken in
 * vocabulary order.
 *
 * What it follows: the paper's section "Speculative Sampling Results"
 * describes the pass in prose -- the target's and the draft's probability
 * outputs on the drafted tokens are compared; a rejection criterion fixes how
 * many drafted tokens are kept; the first rejected token is resampled from a
 * combination of the two distributions and nothing after it is accepted; when
 * every drafted token is accepted one more token is sampled from the target's
 * probabilities.  The paper prints no formula.  The formulas used here are
 * those of the speculative-sampling rule the paper cites for the method:
 *
 *   accept x_i   iff  u_i < p_i(x_i) / q_i(x_i)          (probability min(1, p/q))
 *   on rejection sample from  max(0, p_n - q_n) / sum_j max(0, p_n(j) - q_n(j))
 *   on full acceptance sample from p_K
 *
 * with p = softmax(target_logits / T), q = softmax(draft_logits / T), both
 * samples taken by inverse CDF with the sequence's second uniform u'.
 *
 * Conventions the paper leaves open (each one is a reading, pinned only by
 * the tests that accompany this file, not by the paper):
 *   - strict "<" accepts; evaluated without a division as  u*q < p, so q == 0
 *     with p > 0 accepts and p == q == 0 rejects;
 *   - inverse CDF picks the smallest token id whose inclusive cumulative mass
 *     is strictly above u' * total; if rounding leaves no such id, the largest
 *     id with non-zero mass;
 *   - a residual whose total is zero (impossible in exact arithmetic at a
 *     rejection) falls back to sampling from p_n and raises a status bit;
 *   - one accept uniform per draft position and one resample/bonus uniform per
 *     sequence, stored where the target rows are stored (see below);
 *   - accepted_len counts accepted draft tokens, 0..K_b; K_b = 0 is allowed
 *     and is a plain sample from p_0.
 *
 * Packed layout (ragged lookahead, one K_b per sequence):
 *   off_d[b] = sum_{c<b} max(K_c, 0)      first draft row of sequence b
 *   off_t[b] = off_d[b] + b               first target row of sequence b
 *   target_logits  [n_draft_total + B][ld_target]  row off_t[b]+i, i in [0, K_b]
 *   draft_logits   [n_draft_total    ][ld_draft ]  row off_d[b]+i, i in [0, K_b)
 *   draft_tokens   [n_draft_total]
 *   uniforms       [n_draft_total + B]   entry off_t[b]+i (i < K_b) is u_i,
 *                                        entry off_t[b]+K_b is u'
 *   emitted_tokens [n_draft_total + B]   entries off_t[b] .. off_t[b]+K_b
 *
 * parity status: the accept rule, the residual, the bonus sample, temperature
 * and the packed layout are pinned by tests/test_oracle_*.py (hand-worked
 * cases, exact enumeration of the output distribution, invariants, special
 * cases against numpy routines, a second formulation on random tiny inputs).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1, ORACLE_F16 = 2 };

enum {
    ORACLE_ROW_BAD_K = 1,
    ORACLE_ROW_BAD_TEMPERATURE = 2,
    ORACLE_ROW_BAD_TOKEN = 4,
    ORACLE_ROW_ZERO_RESIDUAL = 8
};

/* IEEE binary16 bits -> double, exactly (subnormals, infinities and NaN included). */
static double half_bits_to_double(uint16_t h)
{
    int sign = h >> 15, e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(1024 + m), e - 25);
    return sign ? -v : v;
}

/* Logit j of a row as a double; fp32, bf16 and fp16 all convert exactly. */
static double logit_at(const void *row, int dtype, int64_t j)
{
    if (dtype == ORACLE_F32)
        return (double)((const float *)row)[j];
    if (dtype == ORACLE_F16)
        return half_bits_to_double(((const uint16_t *)row)[j]);
    uint32_t bits = (uint32_t)((const uint16_t *)row)[j] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static const void *row_ptr(const void *base, int dtype, int64_t row, int64_t ld)
{
    size_t elt = (dtype == ORACLE_F32) ? 4 : 2;
    return (const char *)base + (size_t)row * (size_t)ld * elt;
}

/* Two-pass softmax of logits / T into prob[0..V). */
static void softmax_row(const void *row, int dtype, int64_t V, double T, double *prob)
{
    double m = logit_at(row, dtype, 0);
    for (int64_t j = 1; j < V; ++j) {
        double l = logit_at(row, dtype, j);
        if (l > m) m = l;
    }
    double Z = 0.0;
    for (int64_t j = 0; j < V; ++j) {
        prob[j] = exp((logit_at(row, dtype, j) - m) / T);
        Z += prob[j];
    }
    for (int64_t j = 0; j < V; ++j)
        prob[j] /= Z;
}

/*
 * Inverse CDF over non-negative masses w[0..V) with total W: smallest j whose
 * inclusive cumulative sum is strictly above u*W.  *margin receives the
 * distance, in units of W, from u to the nearer of the two cumulative values
 * that bracket the chosen token (only the upper one for j = 0).
 */
static int32_t inverse_cdf(const double *w, int64_t V, double W, double u, double *margin)
{
    double t = u * W;
    double c = 0.0, c_prev = 0.0;
    int64_t last_nonzero = -1;
    for (int64_t j = 0; j < V; ++j) {
        c_prev = c;
        c += w[j];
        if (w[j] > 0.0) last_nonzero = j;
        if (c > t) {
            double hi = fabs(c / W - u);
            double lo = (j == 0) ? hi : fabs(u - c_prev / W);
            *margin = lo < hi ? lo : hi;
            return (int32_t)j;
        }
    }
    *margin = 0.0; /* u*W not below the rounded total: decided by rounding alone */
    return (int32_t)(last_nonzero < 0 ? V - 1 : last_nonzero);
}

/*
 * Verify sequences b_begin .. b_end-1 of a batch of B.  All pointers are host
 * memory.  Outputs (any of the diagnostic ones may be NULL):
 *   accepted_len [B]                   n_b
 *   emitted_tokens [n_draft_total + B] target packing, -1 padded
 *   row_status [B]                     bit set of ORACLE_ROW_*
 *   p_tok, q_tok, rho [n_draft_total]  p_i(x_i), q_i(x_i), p/q for EVERY draft
 *                                      position, also those after the rejection
 *   accept_margin [n_draft_total]      |u_i - rho_i|
 *   cdf_margin [B]                     margin of the resample / bonus draw
 * Returns 0, or -1 if scratch memory cannot be had.
 */
int oracle_spec_verify(const void *target_logits, const void *draft_logits, int dtype,
                       int64_t V, int64_t ld_target, int64_t ld_draft,
                       const int32_t *draft_tokens, const int32_t *k_per_row,
                       int32_t B, int32_t k_uniform, int64_t n_draft_total,
                       const float *temperature, int temperature_per_row,
                       const float *uniforms,
                       int32_t b_begin, int32_t b_end,
                       int32_t *accepted_len, int32_t *emitted_tokens, int32_t *row_status,
                       double *p_tok, double *q_tok, double *rho,
                       double *accept_margin, double *cdf_margin)
{
    double *p = (double *)malloc(sizeof(double) * (size_t)V);
    double *q = (double *)malloc(sizeof(double) * (size_t)V);
    double *r = (double *)malloc(sizeof(double) * (size_t)V);
    if (!p || !q || !r) {
        free(p); free(q); free(r);
        return -1;
    }

    int64_t off_d = 0;
    for (int32_t b = 0; b < b_end && b < B; ++b) {
        int32_t K_raw = k_per_row ? k_per_row[b] : k_uniform;
        int64_t K = K_raw > 0 ? K_raw : 0;
        int64_t off_t = off_d + b;
        int64_t this_off_d = off_d;
        off_d += K;
        if (b < b_begin) continue;

        int status = 0;
        if (K_raw < 0 || this_off_d + K > n_draft_total) status |= ORACLE_ROW_BAD_K;
        double T = (double)temperature[temperature_per_row ? b : 0];
        if (!(T > 0.0) || isinf(T)) status |= ORACLE_ROW_BAD_TEMPERATURE;
        if (!(status & ORACLE_ROW_BAD_K))
            for (int64_t i = 0; i < K; ++i) {
                int32_t x = draft_tokens[this_off_d + i];
                if (x < 0 || (int64_t)x >= V) status |= ORACLE_ROW_BAD_TOKEN;
            }
        if (status) {
            accepted_len[b] = 0;
            if (this_off_d + K <= n_draft_total) /* the row's slots exist */
                for (int64_t i = 0; i <= K; ++i)
                    emitted_tokens[off_t + i] = -1;
            if (row_status) row_status[b] = status;
            if (cdf_margin) cdf_margin[b] = NAN;
            continue;
        }

        int64_t n = K;        /* first rejected position, K if none */
        int32_t sampled = -1;
        double margin = NAN;
        for (int64_t i = 0; i < K; ++i) {
            softmax_row(row_ptr(target_logits, dtype, off_t + i, ld_target), dtype, V, T, p);
            softmax_row(row_ptr(draft_logits, dtype, this_off_d + i, ld_draft), dtype, V, T, q);
            int32_t x = draft_tokens[this_off_d + i];
            double u = (double)uniforms[off_t + i];
            double ratio = (q[x] > 0.0) ? p[x] / q[x] : (p[x] > 0.0 ? INFINITY : 0.0);
            if (p_tok) p_tok[this_off_d + i] = p[x];
            if (q_tok) q_tok[this_off_d + i] = q[x];
            if (rho) rho[this_off_d + i] = ratio;
            if (accept_margin) accept_margin[this_off_d + i] = fabs(u - ratio);
            int accept = (u * q[x] < p[x]);
            if (!accept && n == K) {
                /* first rejection: resample from the normalised positive part of p - q */
                n = i;
                double R = 0.0;
                for (int64_t j = 0; j < V; ++j) {
                    double d = p[j] - q[j];
                    r[j] = d > 0.0 ? d : 0.0;
                    R += r[j];
                }
                double u2 = (double)uniforms[off_t + K];
                if (R > 0.0) {
                    sampled = inverse_cdf(r, V, R, u2, &margin);
                } else {
                    status |= ORACLE_ROW_ZERO_RESIDUAL;
                    sampled = inverse_cdf(p, V, 1.0, u2, &margin);
                }
                /* later positions are still scored (diagnostics) but decide nothing */
            }
        }
        if (n == K) {
            /* every draft token accepted: bonus token from the last target row */
            softmax_row(row_ptr(target_logits, dtype, off_t + K, ld_target), dtype, V, T, p);
            sampled = inverse_cdf(p, V, 1.0, (double)uniforms[off_t + K], &margin);
        }

        accepted_len[b] = (int32_t)n;
        for (int64_t i = 0; i <= K; ++i) {
            int32_t tok = -1;
            if (i < n) tok = draft_tokens[this_off_d + i];
            else if (i == n) tok = sampled;
            emitted_tokens[off_t + i] = tok;
        }
        if (row_status) row_status[b] = status;
        if (cdf_margin) cdf_margin[b] = margin;
    }

    free(p); free(q); free(r);
    return 0;
}

/*
 * Full probability rows of one (sequence-independent) position, for tests that
 * check distributions: p = softmax(target_row / T), q = softmax(draft_row / T),
 * r = max(0, p - q) (not normalised).  Any output may be NULL; draft_row may be
 * NULL when only p is wanted.
 */
int oracle_position_distributions(const void *target_row, const void *draft_row, int dtype,
                                  int64_t V, double T, double *p_out, double *q_out, double *r_out)
{
    double *p = (double *)malloc(sizeof(double) * (size_t)V);
    double *q = (double *)malloc(sizeof(double) * (size_t)V);
    if (!p || !q) { free(p); free(q); return -1; }
    softmax_row(target_row, dtype, V, T, p);
    if (draft_row) softmax_row(draft_row, dtype, V, T, q);
    for (int64_t j = 0; j < V; ++j) {
        if (p_out) p_out[j] = p[j];
        if (draft_row && q_out) q_out[j] = q[j];
        if (draft_row && r_out) { double d = p[j] - q[j]; r_out[j] = d > 0.0 ? d : 0.0; }
    }
    free(p); free(q);
    return 0;
}

/*
 * Lookahead for the next speculation round, per sequence, from this round's outcome.  The
 * paper argues for speculation whose amount depends on the input (sections "Dynamic Execution"
 * and "Speculative Sampling Results") and gives no rule; the rule stated here is the simple
 * additive one used with assisted generation: if every drafted token was accepted the draft
 * model is doing well on this input, so draft two more next time; otherwise draft one fewer;
 * always within [k_min, k_max].  A heuristic, not part of the sampling rule: it never changes
 * which tokens are emitted.  (parity unpinned by the paper; pinned by hand-worked values.)
 */
void oracle_next_lookahead(const int32_t *k_per_row, int32_t k_uniform, const int32_t *accepted_len,
                           int32_t B, int32_t k_min, int32_t k_max, int32_t *next_k)
{
    for (int32_t b = 0; b < B; ++b) {
        int32_t K = k_per_row ? k_per_row[b] : k_uniform;
        if (K < 0) K = 0;
        int32_t n = accepted_len[b];
        int32_t next = (n >= K) ? K + 2 : K - 1;
        if (next < k_min) next = k_min;
        if (next > k_max) next = k_max;
        next_k[b] = next;
    }
}

/*
 * Greedy verification: the limit T -> 0 of the rule at the top of this file.  Both softmaxes
 * become one-hot at their row's largest logit, the draft token of a position is the draft
 * row's largest logit by construction, and the rule collapses to
 *
 *   accept x_i   iff  x_i == argmax_j target_logits[b,i,j]
 *   at the first mismatch n emit argmax_j target_logits[b,n,:]      (the residual is one-hot there)
 *   with no mismatch emit      argmax_j target_logits[b,K_b,:]      (bonus token)
 *
 * so neither draft logits, temperature nor uniforms are needed.  Reading (the paper does not
 * treat this case): among equal largest logits the smallest token id wins, and a NaN logit is
 * never the largest; a row without any number above -inf yields token 0.
 *
 * Layout, accepted_len, emitted_tokens and row_status as for oracle_spec_verify (status bits
 * ORACLE_ROW_BAD_K and ORACLE_ROW_BAD_TOKEN only).  target_argmax [n_draft_total + B] (may be
 * NULL) receives the argmax of every target row of a valid sequence, in target packing.
 * parity status: pinned by tests/test_oracle_greedy.py (numpy argmax on rows with ties, the
 * stochastic oracle at a temperature close to 0, hand-written cases).
 */
static int32_t argmax_row(const void *row, int dtype, int64_t V)
{
    double m = -INFINITY;
    int64_t arg = 0;
    for (int64_t j = 0; j < V; ++j) {
        double l = logit_at(row, dtype, j);
        if (l > m) { m = l; arg = j; }
    }
    return (int32_t)arg;
}

void oracle_spec_verify_greedy(const void *target_logits, int dtype, int64_t V, int64_t ld_target,
                               const int32_t *draft_tokens, const int32_t *k_per_row,
                               int32_t B, int32_t k_uniform, int64_t n_draft_total,
                               int32_t b_begin, int32_t b_end,
                               int32_t *accepted_len, int32_t *emitted_tokens, int32_t *row_status,
                               int32_t *target_argmax)
{
    int64_t off_d = 0;
    for (int32_t b = 0; b < b_end && b < B; ++b) {
        int32_t K_raw = k_per_row ? k_per_row[b] : k_uniform;
        int64_t K = K_raw > 0 ? K_raw : 0;
        int64_t off_t = off_d + b;
        int64_t this_off_d = off_d;
        off_d += K;
        if (b < b_begin) continue;

        int status = 0;
        if (K_raw < 0 || this_off_d + K > n_draft_total) status |= ORACLE_ROW_BAD_K;
        if (!status)
            for (int64_t i = 0; i < K; ++i) {
                int32_t x = draft_tokens[this_off_d + i];
                if (x < 0 || (int64_t)x >= V) status |= ORACLE_ROW_BAD_TOKEN;
            }
        if (status) {
            accepted_len[b] = 0;
            if (this_off_d + K <= n_draft_total)
                for (int64_t i = 0; i <= K; ++i)
                    emitted_tokens[off_t + i] = -1;
            if (row_status) row_status[b] = status;
            continue;
        }

        int64_t n = K;
        for (int64_t i = 0; i <= K; ++i) {
            int32_t best = argmax_row(row_ptr(target_logits, dtype, off_t + i, ld_target), dtype, V);
            if (target_argmax) target_argmax[off_t + i] = best;
            if (i < n && draft_tokens[this_off_d + i] != best) n = i;   /* first mismatch */
            if (i < n) emitted_tokens[off_t + i] = draft_tokens[this_off_d + i];
            else if (i == n) emitted_tokens[off_t + i] = best;
            else emitted_tokens[off_t + i] = -1;
        }
        accepted_len[b] = (int32_t)n;
        if (row_status) row_status[b] = 0;
    }
}

/*
 * Tree-structured verification.  The paper lists tree drafting among the speculative methods it
 * builds on (section "Speculative Sampling Results": several candidate continuations verified in
 * one target pass) without stating the verification rule; the rule used here is the recursive
 * rejection sampling of those methods, which keeps the emitted tokens distributed exactly as the
 * target's when the children of a context are independent draws from the draft distribution of
 * that context:
 *
 *   at context c (the root, or the context after an accepted node) let r = p_c;
 *   for each child j of c, in increasing node index, with token x_j and uniform u_j:
 *       accept j  iff  u_j < r(x_j) / q_c(x_j)            (evaluated as u_j * q_c(x_j) < r(x_j));
 *       accepted: emit x_j, continue at the context after node j;
 *       rejected: r <- max(0, r - q_c) / sum_v max(0, r(v) - q_c(v))   and try the next child;
 *   when no child is accepted (or c has none) emit one token drawn from r by inverse CDF with
 *   the sequence's last uniform, and stop.
 *
 * A chain (every node the only child of the previous one) is exactly oracle_spec_verify.
 * Readings: a residual that sums to 0 leaves r as it was and raises ORACLE_ROW_ZERO_RESIDUAL;
 * ORACLE_ROW_BAD_PARENT marks a parent index outside [-1, own index).
 *
 * Layout: with N_b nodes per sequence, off_d[b] = sum_{c<b} max(N_c, 0), off_t[b] = off_d[b] + b:
 *   target_logits [n_node_total + B][ld]  row off_t[b] + c: context c (0 = root, j+1 = after node j)
 *   draft_logits  [n_node_total][ld]      row off_d[b] + c: draft distribution of context c, from which
 *                                         its children were drawn; read only if c has children
 *   node_tokens, node_parent [n_node_total]  entry off_d[b] + j; parent -1 = root, else a smaller node index
 *   uniforms [n_node_total + B]           entry off_t[b] + j: u_j of node j; entry off_t[b] + N_b: last uniform
 *   emitted_tokens, accepted_nodes [n_node_total + B]  entries off_t[b] + i: tokens / node indices of the
 *                                         accepted path, then the drawn token (node -1), then -1
 * Diagnostics (may be NULL): p_tok, q_tok [n_node_total]: p_c(x_j), q_c(x_j) of EVERY node j with c its
 * parent's context; walk_margin [B]: smallest |u_j - r(x_j)/q_c(x_j)| over the tests the walk made
 * (+inf if none); cdf_margin [B] as in oracle_spec_verify.
 * parity status: pinned by tests/test_oracle_tree.py (hand-worked cases, equality with
 * oracle_spec_verify on chains, the emitted-token distribution measured by bisection on the
 * uniforms against the target distribution, invariants of the accepted path).
 */
enum { ORACLE_ROW_BAD_PARENT = 32 };

int oracle_spec_verify_tree(const void *target_logits, const void *draft_logits, int dtype,
                            int64_t V, int64_t ld_target, int64_t ld_draft,
                            const int32_t *node_tokens, const int32_t *node_parent,
                            const int32_t *n_per_seq, int32_t B, int32_t n_uniform, int64_t n_node_total,
                            const float *temperature, int temperature_per_seq, const float *uniforms,
                            int32_t b_begin, int32_t b_end,
                            int32_t *accepted_len, int32_t *emitted_tokens, int32_t *accepted_nodes,
                            int32_t *row_status, double *p_tok, double *q_tok,
                            double *walk_margin, double *cdf_margin)
{
    double *p = (double *)malloc(sizeof(double) * (size_t)V);
    double *q = (double *)malloc(sizeof(double) * (size_t)V);
    double *r = (double *)malloc(sizeof(double) * (size_t)V);
    if (!p || !q || !r) { free(p); free(q); free(r); return -1; }

    int64_t off_d = 0;
    for (int32_t b = 0; b < b_end && b < B; ++b) {
        int32_t N_raw = n_per_seq ? n_per_seq[b] : n_uniform;
        int64_t N = N_raw > 0 ? N_raw : 0;
        int64_t d0 = off_d, t0 = off_d + b;
        off_d += N;
        if (b < b_begin) continue;

        int status = 0;
        if (N_raw < 0 || d0 + N > n_node_total) status |= ORACLE_ROW_BAD_K;
        double T = (double)temperature[temperature_per_seq ? b : 0];
        if (!(T > 0.0) || isinf(T)) status |= ORACLE_ROW_BAD_TEMPERATURE;
        if (!(status & ORACLE_ROW_BAD_K))
            for (int64_t j = 0; j < N; ++j) {
                int32_t x = node_tokens[d0 + j], par = node_parent[d0 + j];
                if (x < 0 || (int64_t)x >= V) status |= ORACLE_ROW_BAD_TOKEN;
                if (par < -1 || (int64_t)par >= j) status |= ORACLE_ROW_BAD_PARENT;
            }
        if (status) {
            accepted_len[b] = 0;
            if (d0 + N <= n_node_total)
                for (int64_t i = 0; i <= N; ++i) {
                    emitted_tokens[t0 + i] = -1;
                    if (accepted_nodes) accepted_nodes[t0 + i] = -1;
                }
            if (row_status) row_status[b] = status;
            if (walk_margin) walk_margin[b] = NAN;
            if (cdf_margin) cdf_margin[b] = NAN;
            continue;
        }

        /* probabilities of every node's token under its parent's context (decide nothing) */
        if (p_tok || q_tok)
            for (int64_t c = 0; c < N; ++c) {
                int loaded = 0;
                for (int64_t j = c; j < N; ++j) {
                    if ((int64_t)node_parent[d0 + j] != c - 1) continue;
                    if (!loaded) {
                        softmax_row(row_ptr(target_logits, dtype, t0 + c, ld_target), dtype, V, T, p);
                        softmax_row(row_ptr(draft_logits, dtype, d0 + c, ld_draft), dtype, V, T, q);
                        loaded = 1;
                    }
                    if (p_tok) p_tok[d0 + j] = p[node_tokens[d0 + j]];
                    if (q_tok) q_tok[d0 + j] = q[node_tokens[d0 + j]];
                }
            }

        int64_t c = 0, n = 0;
        int32_t sampled = -1;
        double wmargin = INFINITY, cmargin = NAN;
        for (;;) {
            softmax_row(row_ptr(target_logits, dtype, t0 + c, ld_target), dtype, V, T, r);   /* r = p_c */
            int q_loaded = 0;
            int64_t accepted_node = -1;
            for (int64_t j = c; j < N; ++j) {
                if ((int64_t)node_parent[d0 + j] != c - 1) continue;       /* not a child of this context */
                if (!q_loaded) {
                    softmax_row(row_ptr(draft_logits, dtype, d0 + c, ld_draft), dtype, V, T, q);
                    q_loaded = 1;
                }
                int32_t x = node_tokens[d0 + j];
                double u = (double)uniforms[t0 + j];
                double ratio = (q[x] > 0.0) ? r[x] / q[x] : (r[x] > 0.0 ? INFINITY : 0.0);
                double m = fabs(u - ratio);
                if (m < wmargin) wmargin = m;
                if (u * q[x] < r[x]) { accepted_node = j; break; }
                /* rejected: the residual of r against q_c, renormalised, replaces r */
                double Z = 0.0;
                for (int64_t v = 0; v < V; ++v) {
                    double d = r[v] - q[v];
                    p[v] = d > 0.0 ? d : 0.0;       /* p is free here: used as scratch */
                    Z += p[v];
                }
                if (Z > 0.0)
                    for (int64_t v = 0; v < V; ++v) r[v] = p[v] / Z;
                else
                    status |= ORACLE_ROW_ZERO_RESIDUAL;
            }
            if (accepted_node < 0) {
                double W = 0.0;
                for (int64_t v = 0; v < V; ++v) W += r[v];
                sampled = inverse_cdf(r, V, W, (double)uniforms[t0 + N], &cmargin);
                break;
            }
            emitted_tokens[t0 + n] = node_tokens[d0 + accepted_node];
            if (accepted_nodes) accepted_nodes[t0 + n] = (int32_t)accepted_node;
            ++n;
            c = accepted_node + 1;
        }
        emitted_tokens[t0 + n] = sampled;
        if (accepted_nodes) accepted_nodes[t0 + n] = -1;
        for (int64_t i = n + 1; i <= N; ++i) {
            emitted_tokens[t0 + i] = -1;
            if (accepted_nodes) accepted_nodes[t0 + i] = -1;
        }
        accepted_len[b] = (int32_t)n;
        if (row_status) row_status[b] = status;
        if (walk_margin) walk_margin[b] = wmargin;
        if (cdf_margin) cdf_margin[b] = cmargin;
    }
    free(p); free(q); free(r);
    return 0;
}


/*
 * LM-head product in front of the verify pass (the paper's section "Speculative Sampling Results":
 * the target model scores the drafted positions in one parallel pass; these logits are what the
 * verify pass reads):  logits[r][v] = sum_k hidden[r][k] * weight[v][k], hidden and weight in bf16,
 * the sum taken in double over k in index order, the result rounded once to bf16 (to nearest, ties
 * to even).  Rows r in [r_begin, r_end).  All arrays are bf16 bit patterns.
 * parity status: pinned by tests/test_oracle_lm_head.py (numpy's matmul on exactly representable
 * inputs, hand-checked rounding cases).
 */
static uint16_t double_to_bf16_bits(double x)
{
    float f = (float)x;                 /* not exact in general: handled below */
    /* round the DOUBLE to 8 significant bits directly: scale so that the bf16 ulp is 1 */
    if (x == 0.0 || isnan(x) || isinf(x)) {
        uint32_t b; memcpy(&b, &f, 4); return (uint16_t)(b >> 16);
    }
    int e;
    double m = frexp(fabs(x), &e);       /* |x| = m * 2^e, m in [0.5, 1) */
    if (e < -125) {                      /* bf16 subnormal range: ulp fixed at 2^-133 */
        double q = nearbyint(ldexp(fabs(x), 133));
        double r = ldexp(q, -133);
        f = (float)(x < 0 ? -r : r);
    } else {
        double q = nearbyint(ldexp(m, 8)); /* 8 significant bits, ties to even (default rounding mode) */
        double r = ldexp(q, e - 8);
        f = (float)(x < 0 ? -r : r);     /* exact: r has 8 significant bits */
    }
    uint32_t b; memcpy(&b, &f, 4);
    return (uint16_t)(b >> 16);
}

void oracle_lm_head(const uint16_t *hidden, int64_t ld_h, const uint16_t *weight, int64_t ld_w,
                    int64_t M, int64_t V, int64_t H, int64_t r_begin, int64_t r_end,
                    uint16_t *logits, int64_t ld_out)
{
    (void)M;
    for (int64_t r = r_begin; r < r_end; ++r)
        for (int64_t v = 0; v < V; ++v) {
            double acc = 0.0;
            for (int64_t k = 0; k < H; ++k)
                acc += logit_at(hidden + r * ld_h, ORACLE_BF16, k) * logit_at(weight + v * ld_w, ORACLE_BF16, k);
            logits[r * ld_out + v] = double_to_bf16_bits(acc);
        }
}
