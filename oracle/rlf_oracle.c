/*
 * rlf_oracle.c -- slow, plain fp64 CPU oracle for the GRPO policy-update loss path.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call, link or
 * import this file; it exists so that tests and the benchmark's CPU-baseline
 * leg have a definition-level implementation to compare the GPU kernels with.
 * It shares no code with the CUDA path: no headers, helpers, tables or
 * constants are common to the two.
 *
 * Everything here is the plain definition evaluated in double precision on
 * the input bytes as given (bf16 / fp32 inputs are widened exactly).  There is
 * no blocking, fusion or reordering beyond "one row at a time"; OpenMP only
 * distributes independent rows (or independent output elements) over cores.
 *
 * What the paper fixes and what it leaves open:
 *   - Sec. 2.2 models the trajectory as alternating model-text tokens X and
 *     tool-observation tokens O, and states that observation tokens are
 *     environment output that takes no part in the loss.  Sec. 2.3.2 restates
 *     this as a loss mask over tool results.                -> orc_build_loss_mask
 *   - Sec. 2.3.2 / Fig. 4 name GRPO as the algorithm and Sec. 2.3.1 names the
 *     PPO-style update of the underlying RL trainer, but no formula is printed.
 *     The formulas below are the textbook ones: group-normalised outcome
 *     advantage, clipped importance-ratio surrogate, k3 estimator of the KL
 *     divergence to a reference policy, masked token-mean.
 *                                      -> orc_group_advantage, orc_grpo_loss
 *   - The policy pi_theta(a | s_t) of Sec. 2.2 is a softmax over the
 *     vocabulary; log pi is log-softmax gathered at the sampled token.
 *
 * Parity pins: every function in this file is pinned by tests/test_oracle_*.py
 * (closed forms, brute force, finite differences, library cross-checks).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_BF16 0
#define ORC_F32 1
#define ORC_F64 2

static double widen(const void *base, int dtype, int64_t idx)
{
    if (dtype == ORC_BF16) {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    if (dtype == ORC_F32)
        return (double)((const float *)base)[idx];
    return ((const double *)base)[idx];
}

/*
 * Loss mask over one packed token stream (Sec. 2.2 and Sec. 2.3.2: tool
 * results are excluded from the loss).  An observation span runs from an
 * `open_id` token to the next `close_id` token, both inclusive.  Per sequence
 * b = [cu_seqlens[b], cu_seqlens[b+1]) a two-state machine walks the tokens:
 *     id == open            -> inside := true,  mask 0
 *     inside && id == close -> inside := false, mask 0
 *     otherwise             -> mask = inside ? 0 : 1
 * (a close outside a span is an ordinary token; an open inside a span keeps
 * the span open; an unclosed span runs to the end of its sequence; state never
 * crosses a sequence boundary).  `valid`, if given, is AND-ed in.
 * Outputs: mask[T], seq_id[T] (token -> sequence), *n_out = sum of mask.
 */
int orc_build_loss_mask(const int32_t *ids, const int32_t *cu_seqlens, int32_t B, int64_t T,
                        int32_t open_id, int32_t close_id, const uint8_t *valid,
                        uint8_t *mask, int32_t *seq_id, int64_t *n_out)
{
    int64_t n = 0;
    for (int64_t t = 0; t < T; ++t) {
        mask[t] = 0;
        if (seq_id) seq_id[t] = -1;
    }
    for (int32_t b = 0; b < B; ++b) {
        int inside = 0;
        for (int64_t t = cu_seqlens[b]; t < cu_seqlens[b + 1]; ++t) {
            if (t < 0 || t >= T) return -2;
            uint8_t m;
            if (ids[t] == open_id) {
                inside = 1;
                m = 0;
            } else if (inside && ids[t] == close_id) {
                inside = 0;
                m = 0;
            } else {
                m = inside ? 0 : 1;
            }
            if (valid && !valid[t]) m = 0;
            mask[t] = m;
            if (seq_id) seq_id[t] = b;
            n += m;
        }
    }
    *n_out = n;
    return 0;
}

/*
 * Group-relative outcome advantage (GRPO, named in Sec. 2.3.2 / Fig. 4):
 *     A_i = (r_i - mean_g) / (std_g + eps),   g = group of response i.
 * std uses divisor n-1 when `unbiased` (n = group size) and n otherwise; a
 * group of one response, or one with zero spread, gets A = 0 (numerator 0;
 * with eps = 0 the quotient 0/0 is read as 0 too) -- for n = 1 with the
 * unbiased divisor std is defined as 0.
 * group_id == NULL means contiguous groups of `g_or_num_groups` responses.
 */
int orc_group_advantage(const float *rewards, const int32_t *group_id, int32_t B,
                        int32_t g_or_num_groups, double eps, int unbiased, double *adv)
{
    int32_t num_groups;
    if (group_id) {
        num_groups = g_or_num_groups;
    } else {
        if (g_or_num_groups <= 0) return -2;
        num_groups = (B + g_or_num_groups - 1) / g_or_num_groups;
    }
    for (int32_t g = 0; g < num_groups; ++g) {
        double sum = 0.0;
        int64_t n = 0;
        for (int32_t i = 0; i < B; ++i) {
            int32_t gi = group_id ? group_id[i] : i / g_or_num_groups;
            if (gi == g) { sum += (double)rewards[i]; ++n; }
        }
        if (n == 0) continue;
        double mean = sum / (double)n;
        double ss = 0.0;
        for (int32_t i = 0; i < B; ++i) {
            int32_t gi = group_id ? group_id[i] : i / g_or_num_groups;
            if (gi == g) { double d = (double)rewards[i] - mean; ss += d * d; }
        }
        double div = unbiased ? (double)(n - 1) : (double)n;
        double sd = (div > 0.0) ? sqrt(ss / div) : 0.0;
        for (int32_t i = 0; i < B; ++i) {
            int32_t gi = group_id ? group_id[i] : i / g_or_num_groups;
            /* a group without spread carries no signal: A = 0 also when eps = 0 (0/0 otherwise) */
            if (gi == g) adv[i] = (sd + eps > 0.0) ? ((double)rewards[i] - mean) / (sd + eps) : 0.0;
        }
    }
    if (group_id)
        for (int32_t i = 0; i < B; ++i)
            if (group_id[i] < 0 || group_id[i] >= num_groups) return -2;
    return 0;
}

/* Per-token loss terms given the token's log-prob under the current policy.
 *   rho = exp(logp - old);  pg = -min(rho*A, clip(rho, 1-e, 1+e)*A)
 *   d = ref - logp;         kl = exp(d) - d - 1          (k3 estimator)
 *   dpg/dlogp = 0 when the clipped branch is the active minimum
 *               (A>0 and rho>1+e, or A<0 and rho<1-e), else -A*rho
 *   dkl/dlogp = 1 - exp(d)
 */
static void token_terms_lohi(double logp, double old_lp, double ref_lp, double A, double lo, double hi,
                             double *pg, double *kl, double *dpg, double *dkl, int *clipped)
{
    double rho = exp(logp - old_lp);
    double rc = rho < lo ? lo : (rho > hi ? hi : rho);
    double s1 = rho * A, s2 = rc * A;
    *pg = -(s1 < s2 ? s1 : s2);
    *clipped = (A > 0.0 && rho > hi) || (A < 0.0 && rho < lo);
    *dpg = *clipped ? 0.0 : -A * rho;
    double d = ref_lp - logp;
    *kl = exp(d) - d - 1.0;
    *dkl = 1.0 - exp(d);
}

static void token_terms(double logp, double old_lp, double ref_lp, double A, double eps_clip,
                        double *pg, double *kl, double *dpg, double *dkl, int *clipped)
{
    token_terms_lohi(logp, old_lp, ref_lp, A, 1.0 - eps_clip, 1.0 + eps_clip, pg, kl, dpg, dkl, clipped);
}

/* log-softmax statistics of one row: m = max_v z, and log s with s = sum_v exp(z - m), so that
 * lse = m + log s.  The two parts are returned separately and every use below subtracts m from a
 * logit FIRST, (z - m) - log s: the same quantity as z - lse, but it keeps full precision when
 * |m| is so large that m + log s would absorb log s. */
static void row_stats(const void *logits, int dtype, int64_t off, int32_t V, double *m_out, double *logs_out)
{
    double m = -INFINITY;
    for (int32_t v = 0; v < V; ++v) {
        double z = widen(logits, dtype, off + v);
        if (z > m) m = z;
    }
    double s = 0.0;
    for (int32_t v = 0; v < V; ++v)
        s += exp(widen(logits, dtype, off + v) - m);
    *m_out = m;
    *logs_out = log(s);
}

/*
 * GRPO loss over materialised logits, forward and backward.
 *   row t:  lse_t = log sum_v exp z[t,v];  logp_t = z[t, ids[t]] - lse_t
 *   l_t = pg_t + beta * kl_t   (token_terms above, A = adv[seq_id[t]])
 *   N = denom if denom >= 0 else sum_t mask_t;   Nd = max(N, 1)
 *   loss[0] = sum_t mask_t l_t / Nd      loss[1] = sum mask pg / Nd
 *   loss[2] = sum mask kl / Nd           loss[3] = sum mask clipped / Nd
 *   grad[t,v] = d loss[0] / d z[t,v]
 *             = (mask_t / Nd) (dpg_t + beta dkl_t) (1[v = ids[t]] - p[t,v]),  p = softmax(z[t,:])
 * logp is produced for every row, masked or not.  grad may be NULL.
 * coef_out (nullable) receives c_t with grad[t,v] = c_t (p[t,v] - 1[v=y]).
 */
int orc_grpo_loss(const void *logits, int dtype, int64_t T, int32_t V, int64_t row_stride,
                  const int32_t *ids, const int32_t *seq_id, const float *adv,
                  const float *old_logp, const float *ref_logp, const uint8_t *mask,
                  double eps_clip, double beta_kl, int64_t denom,
                  double *logp_out, double *loss_out, double *grad, double *coef_out)
{
    int64_t n = 0;
    for (int64_t t = 0; t < T; ++t) n += mask[t] ? 1 : 0;
    if (denom >= 0) n = denom;
    double nd = n > 1 ? (double)n : 1.0;

    double *pg_t = (double *)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
    double *kl_t = (double *)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
    uint8_t *cl_t = (uint8_t *)malloc((size_t)(T > 0 ? T : 1));
    if (!pg_t || !kl_t || !cl_t) return -7;
    int bad = 0;

#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t t = 0; t < T; ++t) {
        int64_t off = t * row_stride;
        int32_t y = ids[t];
        if (y < 0 || y >= V) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        double m, logs;
        row_stats(logits, dtype, off, V, &m, &logs);
        double logp = (widen(logits, dtype, off + y) - m) - logs;
        logp_out[t] = logp;
        double A = (double)adv[seq_id[t]];
        double pg, kl, dpg, dkl;
        int clipped;
        token_terms(logp, (double)old_logp[t], (double)ref_logp[t], A, eps_clip,
                    &pg, &kl, &dpg, &dkl, &clipped);
        pg_t[t] = pg;
        kl_t[t] = kl;
        cl_t[t] = (uint8_t)clipped;
        double w = mask[t] ? 1.0 / nd : 0.0;
        double g = w * (dpg + beta_kl * dkl); /* d loss / d logp_t */
        if (coef_out) coef_out[t] = -g;
        if (grad) {
            for (int32_t v = 0; v < V; ++v) {
                double p = exp((widen(logits, dtype, off + v) - m) - logs);
                grad[t * (int64_t)V + v] = g * ((v == y ? 1.0 : 0.0) - p);
            }
        }
    }
    if (bad) { free(pg_t); free(kl_t); free(cl_t); return -2; }

    double s_pg = 0.0, s_kl = 0.0, s_cl = 0.0;
    for (int64_t t = 0; t < T; ++t) {
        if (!mask[t]) continue;
        s_pg += pg_t[t];
        s_kl += kl_t[t];
        s_cl += (double)cl_t[t];
    }
    loss_out[0] = (s_pg + beta_kl * s_kl) / nd;
    loss_out[1] = s_pg / nd;
    loss_out[2] = s_kl / nd;
    loss_out[3] = s_cl / nd;
    free(pg_t); free(kl_t); free(cl_t);
    return 0;
}

/*
 * Objective variants of orc_grpo_loss (the paper names GRPO / a PPO-style update in Sec. 2.3 and
 * prints no objective; these are the common alternatives to the symmetric-clip token mean):
 *   - asymmetric clip range: clip(rho, 1 - eps_low, 1 + eps_high);
 *   - aggregation 0: masked token mean, weight w_t = mask_t / max(N, 1), N = denom or sum of mask;
 *     aggregation 1: mean over sequences of each sequence's masked token mean,
 *         w_t = mask_t / (n_b * max(S, 1)),  n_b = sum of mask in the sequence b of token t,
 *         S = denom if denom >= 0 else the number of sequences with n_b > 0.
 *   loss_out[k] = sum_t w_t x_t for x in {pg + beta kl, pg, kl, clipped};
 *   grad[t,v] = w_t (dpg_t + beta dkl_t) (1[v = y_t] - p[t,v]).
 * num_seqs = number of sequences (seq_id values lie in [0, num_seqs)).
 */
int orc_grpo_loss_obj(const void *logits, int dtype, int64_t T, int32_t V, int64_t row_stride,
                      const int32_t *ids, const int32_t *seq_id, const float *adv, int32_t num_seqs,
                      const float *old_logp, const float *ref_logp, const uint8_t *mask,
                      double eps_low, double eps_high, double beta_kl, int aggregation, int64_t denom,
                      double *logp_out, double *loss_out, double *grad, double *coef_out)
{
    double *w = (double *)calloc((size_t)(T > 0 ? T : 1), sizeof(double));
    int64_t *nb = (int64_t *)calloc((size_t)(num_seqs > 0 ? num_seqs : 1), sizeof(int64_t));
    if (!w || !nb) return -7;
    for (int64_t t = 0; t < T; ++t) {
        if (seq_id[t] < 0 || seq_id[t] >= num_seqs) { free(w); free(nb); return -2; }
        if (mask[t]) nb[seq_id[t]] += 1;
    }
    if (aggregation == 0) {
        int64_t n = 0;
        for (int32_t b = 0; b < num_seqs; ++b) n += nb[b];
        if (denom >= 0) n = denom;
        double nd = n > 1 ? (double)n : 1.0;
        for (int64_t t = 0; t < T; ++t) w[t] = mask[t] ? 1.0 / nd : 0.0;
    } else {
        int64_t S = 0;
        for (int32_t b = 0; b < num_seqs; ++b) S += nb[b] > 0 ? 1 : 0;
        if (denom >= 0) S = denom;
        double sd = S > 1 ? (double)S : 1.0;
        for (int64_t t = 0; t < T; ++t) w[t] = mask[t] ? 1.0 / ((double)nb[seq_id[t]] * sd) : 0.0;
    }
    double *terms = (double *)calloc((size_t)(T > 0 ? T : 1) * 3, sizeof(double));
    if (!terms) { free(w); free(nb); return -7; }
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t t = 0; t < T; ++t) {
        int64_t off = t * row_stride;
        int32_t y = ids[t];
        if (y < 0 || y >= V) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        double m, logs;
        row_stats(logits, dtype, off, V, &m, &logs);
        double logp = (widen(logits, dtype, off + y) - m) - logs;
        logp_out[t] = logp;
        double pg, kl, dpg, dkl;
        int clipped;
        token_terms_lohi(logp, (double)old_logp[t], (double)ref_logp[t], (double)adv[seq_id[t]],
                         1.0 - eps_low, 1.0 + eps_high, &pg, &kl, &dpg, &dkl, &clipped);
        terms[3 * t] = pg;
        terms[3 * t + 1] = kl;
        terms[3 * t + 2] = (double)clipped;
        double g = w[t] * (dpg + beta_kl * dkl);
        if (coef_out) coef_out[t] = -g;
        if (grad) {
            for (int32_t v = 0; v < V; ++v) {
                double p = exp((widen(logits, dtype, off + v) - m) - logs);
                grad[t * (int64_t)V + v] = g * ((v == y ? 1.0 : 0.0) - p);
            }
        }
    }
    double s_pg = 0.0, s_kl = 0.0, s_cl = 0.0;
    for (int64_t t = 0; t < T; ++t) {
        s_pg += w[t] * terms[3 * t];
        s_kl += w[t] * terms[3 * t + 1];
        s_cl += w[t] * terms[3 * t + 2];
    }
    loss_out[0] = s_pg + beta_kl * s_kl;
    loss_out[1] = s_pg;
    loss_out[2] = s_kl;
    loss_out[3] = s_cl;
    free(w); free(nb); free(terms);
    return bad ? -2 : 0;
}

/*
 * Fused LM-head variant: the logits are z[t,v] = sum_k H[t,k] W[v,k] (bf16
 * inputs widened to fp64, fp64 products and sums), then exactly orc_grpo_loss
 * on those fp64 logits, then the chain rule through the contraction:
 *   grad_hidden[t,k] = sum_v grad_z[t,v] W[v,k]
 *   grad_W[v,k]      = sum_t grad_z[t,v] H[t,k]
 * Materialises z and grad_z as [T,V] fp64: for small T only.
 * grad_hidden / grad_W may be NULL (skipped).  z_out (nullable) gets z.
 */
/* z[t,v] = sum_k H[t,k] W[v,k], every product and sum in fp64 */
static void head_logits(const uint16_t *hidden, const uint16_t *W, int64_t T, int32_t D, int32_t V, double *z)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t t = 0; t < T; ++t)
        for (int32_t v = 0; v < V; ++v) {
            double acc = 0.0;
            for (int32_t k = 0; k < D; ++k)
                acc += widen(hidden, ORC_BF16, t * (int64_t)D + k) *
                       widen(W, ORC_BF16, v * (int64_t)D + k);
            z[t * (int64_t)V + v] = acc;
        }
}

/* chain rule through the contraction, given grad_z = gz */
static void head_backward(const uint16_t *hidden, const uint16_t *W, int64_t T, int32_t D, int32_t V,
                          const double *gz, double *grad_hidden, double *grad_W)
{
    if (grad_hidden) {
#pragma omp parallel for schedule(dynamic, 1)
        for (int64_t t = 0; t < T; ++t)
            for (int32_t k = 0; k < D; ++k) {
                double acc = 0.0;
                for (int32_t v = 0; v < V; ++v)
                    acc += gz[t * (int64_t)V + v] * widen(W, ORC_BF16, v * (int64_t)D + k);
                grad_hidden[t * (int64_t)D + k] = acc;
            }
    }
    if (grad_W) {
#pragma omp parallel for schedule(dynamic, 16)
        for (int32_t v = 0; v < V; ++v)
            for (int32_t k = 0; k < D; ++k) {
                double acc = 0.0;
                for (int64_t t = 0; t < T; ++t)
                    acc += gz[t * (int64_t)V + v] * widen(hidden, ORC_BF16, t * (int64_t)D + k);
                grad_W[v * (int64_t)D + k] = acc;
            }
    }
}

int orc_fused_lmhead_grpo(const uint16_t *hidden, const uint16_t *W, int64_t T, int32_t D,
                          int32_t V, const int32_t *ids, const int32_t *seq_id,
                          const float *adv, const float *old_logp, const float *ref_logp,
                          const uint8_t *mask, double eps_clip, double beta_kl, int64_t denom,
                          double *logp_out, double *loss_out, double *grad_hidden,
                          double *grad_W, double *z_out)
{
    size_t tv = (size_t)(T > 0 ? T : 1) * (size_t)V;
    double *z = z_out ? z_out : (double *)malloc(sizeof(double) * tv);
    int need_g = grad_hidden || grad_W;
    double *gz = need_g ? (double *)malloc(sizeof(double) * tv) : NULL;
    if (!z || (need_g && !gz)) return -7;

    head_logits(hidden, W, T, D, V, z);
    int rc = orc_grpo_loss(z, ORC_F64, T, V, V, ids, seq_id, adv, old_logp, ref_logp, mask,
                           eps_clip, beta_kl, denom, logp_out, loss_out, gz, NULL);
    if (rc == 0)
        head_backward(hidden, W, T, D, V, gz, grad_hidden, grad_W);
    if (!z_out) free(z);
    free(gz);
    return rc;
}

/*
 * The fused LM-head variant under the objective variants: the same fp64 logits, then exactly
 * orc_grpo_loss_obj on them (asymmetric clip range, token-mean or sequence-mean aggregation), then
 * the same chain rule through the contraction.
 */
int orc_fused_lmhead_grpo_obj(const uint16_t *hidden, const uint16_t *W, int64_t T, int32_t D,
                              int32_t V, const int32_t *ids, const int32_t *seq_id,
                              const float *adv, int32_t num_seqs, const float *old_logp,
                              const float *ref_logp, const uint8_t *mask, double eps_low,
                              double eps_high, double beta_kl, int aggregation, int64_t denom,
                              double *logp_out, double *loss_out, double *grad_hidden, double *grad_W)
{
    size_t tv = (size_t)(T > 0 ? T : 1) * (size_t)V;
    double *z = (double *)malloc(sizeof(double) * tv);
    int need_g = grad_hidden || grad_W;
    double *gz = need_g ? (double *)malloc(sizeof(double) * tv) : NULL;
    if (!z || (need_g && !gz)) return -7;

    head_logits(hidden, W, T, D, V, z);
    int rc = orc_grpo_loss_obj(z, ORC_F64, T, V, V, ids, seq_id, adv, num_seqs, old_logp, ref_logp, mask,
                               eps_low, eps_high, beta_kl, aggregation, denom, logp_out, loss_out, gz, NULL);
    if (rc == 0)
        head_backward(hidden, W, T, D, V, gz, grad_hidden, grad_W);
    free(z);
    free(gz);
    return rc;
}

/*
 * Forward-only log-prob and entropy of each row's softmax (the behaviour / reference policy pass that
 * produces old_logp and ref_logp for the PPO-style update of Sec. 2.3.1; the policy of Sec. 2.2):
 *     logp_t = z[t, y_t] - lse_t
 *     H_t    = - sum_v p_v log p_v,   p_v = exp(z_v - lse_t),   a term with p_v = 0 counts 0
 * entropy_out may be NULL.
 */
int orc_logp_entropy(const void *logits, int dtype, int64_t T, int32_t V, int64_t row_stride,
                     const int32_t *ids, double *logp_out, double *entropy_out)
{
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t t = 0; t < T; ++t) {
        int64_t off = t * row_stride;
        int32_t y = ids[t];
        if (y < 0 || y >= V) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        double m, logs;
        row_stats(logits, dtype, off, V, &m, &logs);
        logp_out[t] = (widen(logits, dtype, off + y) - m) - logs;
        if (entropy_out) {
            double h = 0.0;
            for (int32_t v = 0; v < V; ++v) {
                double lp = (widen(logits, dtype, off + v) - m) - logs;   /* log p_v */
                double pv = exp(lp);
                if (pv > 0.0) h -= pv * lp;
            }
            entropy_out[t] = h;
        }
    }
    return bad ? -2 : 0;
}

/*
 * Forward-only log-prob and entropy with the logits formed from the head: z = H W^T in fp64
 * (head_logits), then exactly orc_logp_entropy on them.  entropy_out may be NULL.
 */
int orc_fused_lmhead_logp_entropy(const uint16_t *hidden, const uint16_t *W, int64_t T, int32_t D, int32_t V,
                                  const int32_t *ids, double *logp_out, double *entropy_out)
{
    double *z = (double *)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1) * (size_t)V);
    if (!z) return -7;
    head_logits(hidden, W, T, D, V, z);
    int rc = orc_logp_entropy(z, ORC_F64, T, V, V, ids, logp_out, entropy_out);
    free(z);
    return rc;
}

/* Rule reward, Eq. 1: R = sum_i w_i r_i over n rule scores, for each of B responses.
 * scores is [B, n] row-major. */
int orc_rule_reward(const float *scores, const float *weights, int32_t B, int32_t n, double *R)
{
    for (int32_t b = 0; b < B; ++b) {
        double acc = 0.0;
        for (int32_t i = 0; i < n; ++i)
            acc += (double)weights[i] * (double)scores[b * (int64_t)n + i];
        R[b] = acc;
    }
    return 0;
}

/*
 * KL penalty folded into the reward instead of the loss (an objective variant; the paper names
 * GRPO / a PPO-style update in Sec. 2.3 and prints no formula, so this is the common form of the
 * RL trainers it builds on): the outcome reward of response b is reduced by beta times the summed
 * per-token divergence estimate between the behaviour policy and the reference policy over the
 * response's loss-carrying tokens,
 *     R'_b = R_b - beta * sum_{t in b} mask_t k(old_logp_t, ref_logp_t),   d = old_logp_t - ref_logp_t
 *     kind 0 (k1): k = d        kind 1 (k2): k = d^2 / 2        kind 2 (k3): k = exp(-d) + d - 1
 * kl_seq[b] (optional) receives the summed estimate itself.  Tokens outside every response count
 * for nothing.  Returns -3 for an unknown kind, -2 for a malformed cu_seqlens.
 */
int orc_kl_in_reward(const float *rewards, const float *old_logp, const float *ref_logp, const uint8_t *mask,
                     const int32_t *cu_seqlens, int32_t B, int64_t T, double beta, int kind,
                     double *reward_out, double *kl_seq)
{
    if (kind < 0 || kind > 2)
        return -3;
    for (int32_t b = 0; b < B; ++b) {
        int64_t lo = cu_seqlens[b], hi = cu_seqlens[b + 1];
        if (lo < 0 || hi < lo || hi > T)
            return -2;
        double acc = 0.0;
        for (int64_t t = lo; t < hi; ++t) {
            if (!mask[t])
                continue;
            double d = (double)old_logp[t] - (double)ref_logp[t];
            double k;
            if (kind == 0)
                k = d;
            else if (kind == 1)
                k = 0.5 * d * d;
            else
                k = exp(-d) + d - 1.0;
            acc += k;
        }
        if (kl_seq)
            kl_seq[b] = acc;
        reward_out[b] = (double)rewards[b] - beta * acc;
    }
    return 0;
}

int orc_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}
