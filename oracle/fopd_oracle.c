/*
 * fopd_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of what the f-OPD loss path computes,
 * written from the paper's definitions.  It exists so that the CUDA library
 * can be checked against something independent: it shares no code, header,
 * table or helper with the CUDA sources and must only ever be called from
 * the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * Every function below cites the passage of the paper it evaluates.  All
 * arithmetic is double precision; logits arrive as bf16 or fp32 bit patterns
 * and are widened exactly.  Rows are independent, so the only "optimisation"
 * is an OpenMP loop over rows.  Natural logarithms throughout.
 *
 * Readings of the paper taken here (the paper leaves them open):
 *   - the token loss l(p, q) of Eq. 12 is the full-vocabulary reverse KL,
 *     KL(student || teacher);
 *   - the rollout drift KL(pi^t || pi^r) of Eq. 10 (first row) is estimated
 *     from the stored token y ~ pi^r alone by  k3(rho) = rho*log(rho) - rho + 1
 *     with rho = pi^t(y)/pi^r(y), whose expectation under pi^r is that KL;
 *   - the rollout-aligned set U^roll is the rows with mask = 1; the supervision
 *     diagnostics (oracle_row_divergence) take their own mask U^sup, and the
 *     loss path uses one set for both;
 *   - the gate w_i = ReLU(f_i - xi) is a constant in the backward pass;
 *   - the batch mean of Eq. 16 / Algorithm 1 divides by the number of samples
 *     passed in, gated and invalid ones included;
 *   - the sampled-token form of the token loss (the setup Sec. 5 says the
 *     experiments follow, and the sampled-token objectives of Appendix B) is
 *     rho_n (log p_s(y_n) - log p_t(y_n)) on the stored token y_n ~ pi^r, with
 *     rho_n = pi^t(y_n) / pi^r(y_n): its expectation under pi^r is the
 *     full-vocabulary reverse KL of Eq. 12.  In its gradient the importance
 *     ratio carries the derivative and the log-ratio is a constant (the reward
 *     of a policy-gradient step), whose expectation under pi^r is the gradient
 *     of that KL.
 *
 * Pins (tests/test_oracle_pins.py): every function here is pinned to closed
 * forms, brute force on tiny vocabularies, library routines in float64,
 * identities and central finite differences; none is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#define ORACLE_BF16 0
#define ORACLE_F32 1

/* Exact widening of one stored logit to double. */
static double logit_at(const void *base, int dtype, int64_t idx) {
    if (dtype == ORACLE_BF16) {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float *)base)[idx];
}

/* log sum_v exp(z_v) of one row: the normaliser of the softmax policy
 * pi(. | x) that Sec. 3.1 works with.  Max-shifted for range only. */
static double row_logsumexp(const void *row, int dtype, int64_t V) {
    double m = -INFINITY;
    for (int64_t v = 0; v < V; ++v) {
        double z = logit_at(row, dtype, v);
        if (z > m) m = z;
    }
    double s = 0.0;
    for (int64_t v = 0; v < V; ++v) s += exp(logit_at(row, dtype, v) - m);
    return m + log(s);
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n) {
#ifdef _OPENMP
    extern void omp_set_num_threads(int);
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/*
 * Per-token quantities of one chunk of rows.
 *
 *   lse_s, lse_t : log-normalisers of the student and teacher rows
 *   lp_s,  lp_t  : log-probabilities of the stored token y_n (Sec. 4.1: the
 *                  buffer keeps the generated tokens y_{i,h})
 *   kl           : token loss of Eq. 12 under the reverse-KL reading,
 *                  sum_v p_s(v) (log p_s(v) - log p_t(v))
 *   d, rho, k3   : d = lp_s - b_n, rho = exp(d) = pi^t(y)/pi^r(y), and the
 *                  per-token integrand of D_roll (Eq. 10, first row)
 *   valid        : 1 where the row counts (mask = 1, ids in range)
 *
 * A row with mask = 0, a token outside [0, V) or a sample id outside [0, B)
 * is not aligned: every output of it is 0 and valid = 0.
 */
void oracle_token_stats(const void *student, const void *teacher, int dtype,
                        int64_t n_rows, int64_t V, int64_t row_stride,
                        const int32_t *tokens, const float *behav_logprob,
                        const uint8_t *mask, const int32_t *sample_id, int32_t B,
                        double *lse_s, double *lse_t, double *lp_s, double *lp_t,
                        double *kl, double *d, double *rho, double *k3,
                        uint8_t *valid) {
    size_t esz = dtype == ORACLE_BF16 ? 2 : 4;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t n = 0; n < n_rows; ++n) {
        int ok = mask[n] != 0 && tokens[n] >= 0 && tokens[n] < V &&
                 sample_id[n] >= 0 && sample_id[n] < B;
        valid[n] = (uint8_t)ok;
        if (!ok) {
            lse_s[n] = lse_t[n] = lp_s[n] = lp_t[n] = 0.0;
            kl[n] = d[n] = rho[n] = k3[n] = 0.0;
            continue;
        }
        const void *srow = (const char *)student + (size_t)n * row_stride * esz;
        const void *trow = (const char *)teacher + (size_t)n * row_stride * esz;
        double ls = row_logsumexp(srow, dtype, V);
        double lt = row_logsumexp(trow, dtype, V);
        double acc = 0.0;
        for (int64_t v = 0; v < V; ++v) {
            double logp = logit_at(srow, dtype, v) - ls;
            double logq = logit_at(trow, dtype, v) - lt;
            acc += exp(logp) * (logp - logq);
        }
        lse_s[n] = ls;
        lse_t[n] = lt;
        lp_s[n] = logit_at(srow, dtype, tokens[n]) - ls;
        lp_t[n] = logit_at(trow, dtype, tokens[n]) - lt;
        kl[n] = acc;
        double dn = lp_s[n] - (double)behav_logprob[n];
        d[n] = dn;
        rho[n] = exp(dn);
        /* rho*log(rho) - (rho - 1); expm1 keeps the second term exact near 0 */
        k3[n] = exp(dn) * dn - expm1(dn);
    }
}

/*
 * Sums over the aligned rows of each sample (the numerators and |U_i| of
 * Eq. 10 and Eq. 12).  acc is [B,3] = {count, sum k3, sum kl} and is ADDED
 * to, so a sample that spans several chunks accumulates across calls.
 */
void oracle_sample_accumulate(int64_t n_rows, int32_t B, const int32_t *sample_id,
                              const uint8_t *valid, const double *kl,
                              const double *k3, double *acc) {
    (void)B;
    for (int64_t n = 0; n < n_rows; ++n) {
        if (!valid[n]) continue;
        double *a = acc + 3 * (size_t)sample_id[n];
        a[0] += 1.0;
        a[1] += k3[n];
        a[2] += kl[n];
    }
}

/*
 * Per-sample freshness and gate.
 *   D_roll_i = sum k3 / |U_i|,  l_i = sum kl / |U_i|            (Eq. 10, Eq. 12)
 *   f_i = exp(-alpha sqrt(D_roll_i) - beta sqrt(D_sup_i)) / (tau_i + 1)  (Eq. 11)
 *   w_i = max(f_i - xi, 0)                                 (Eq. 13, sigma = ReLU)
 *   m_i = |U_i| / H_i                                      (Algorithm 1)
 *   coef_i = w_i / (B |U_i|): the weight of one token's loss in Eq. 16
 * A sample with no aligned row, H_i <= 0 or tau_i < 0 is invalid: f = w = m =
 * coef = 0 (Algorithm 1, the |U| = 0 branch).  d_sup may be NULL (all zero:
 * teacher and context unchanged, Appendix remark on supervision drift).
 */
void oracle_sample_freshness(int32_t B, const double *acc, const int32_t *tau,
                             const int32_t *H, const float *d_sup, double alpha,
                             double beta, double xi, double *f, double *w,
                             double *D_roll, double *ell, double *m,
                             double *coef, uint8_t *valid) {
    for (int32_t i = 0; i < B; ++i) {
        double cnt = acc[3 * i];
        /* d_sup = +inf stands for an empty supervision-aligned set: Algorithm 1
         * marks such a sample invalid exactly like an empty rollout-aligned set. */
        int ok = cnt > 0.0 && H[i] > 0 && tau[i] >= 0 && !(d_sup && isinf(d_sup[i]));
        valid[i] = (uint8_t)ok;
        if (!ok) {
            f[i] = w[i] = D_roll[i] = ell[i] = m[i] = coef[i] = 0.0;
            continue;
        }
        D_roll[i] = acc[3 * i + 1] / cnt;
        ell[i] = acc[3 * i + 2] / cnt;
        double ds = d_sup ? (double)d_sup[i] : 0.0;
        double droll_pos = D_roll[i] > 0.0 ? D_roll[i] : 0.0;
        double surrogate = alpha * sqrt(droll_pos) + beta * sqrt(ds > 0.0 ? ds : 0.0);
        f[i] = exp(-surrogate) / ((double)tau[i] + 1.0);
        double g = f[i] - xi;
        w[i] = g > 0.0 ? g : 0.0;
        m[i] = cnt / (double)H[i];
        coef[i] = w[i] / ((double)B * cnt);
    }
}

/*
 * Row-wise KL(p || q) and entropy H(p) for p = softmax(first[n,:]),
 * q = softmax(second[n,:]) at rows with mask = 1 (zeros elsewhere).  With the
 * teacher's logits under the current and under the stored context this is the
 * integrand of the supervision drift D_sup, Eq. 10 second row; the entropy is
 * the response-entropy monitoring signal of Appendix B.
 */
void oracle_row_divergence(const void *first, const void *second, int dtype,
                           int64_t n_rows, int64_t V, int64_t stride,
                           const uint8_t *mask, double *kl, double *entropy) {
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t n = 0; n < n_rows; ++n) {
        kl[n] = entropy[n] = 0.0;
        if (!mask[n]) continue;
        size_t esz = dtype == ORACLE_BF16 ? 2 : 4;
        const char *a = (const char *)first + (size_t)n * stride * esz;
        const char *b = (const char *)second + (size_t)n * stride * esz;
        double la = row_logsumexp(a, dtype, V), lb = row_logsumexp(b, dtype, V);
        double k = 0.0, h = 0.0;
        for (int64_t v = 0; v < V; ++v) {
            double lp = logit_at(a, dtype, v) - la, lq = logit_at(b, dtype, v) - lb;
            double p = exp(lp);
            k += p * (lp - lq);
            h -= p * lp;
        }
        kl[n] = k;
        entropy[n] = h;
    }
}

/* Objective of Eq. 16 as Algorithm 1 forms it on a minibatch:
 * L_i = w_i (l_i + lambda D_roll_i),  L = (1/B) sum_i L_i. */
double oracle_loss(int32_t B, const double *w, const double *ell,
                   const double *D_roll, double lambda, double *per_sample) {
    double total = 0.0;
    for (int32_t i = 0; i < B; ++i) {
        double Li = w[i] * (ell[i] + lambda * D_roll[i]);
        if (per_sample) per_sample[i] = Li;
        total += Li;
    }
    return total / (double)B;
}

/*
 * Gradient of L with respect to the student logits of selected rows, with
 * w_i held constant.  For an aligned row n of sample i and c = coef_i:
 *
 *   d kl_n / dS_v = p_s(v) [ (log p_s(v) - log p_t(v)) - kl_n ]
 *   d k3_n / dS_v = rho_n d_n ( 1[v = y_n] - p_s(v) )     (d k3/dd = rho d)
 *   dS[n, v]      = c ( d kl_n/dS_v + lambda d k3_n/dS_v )
 *
 * Rows that are not aligned, or whose sample has coef = 0, get zeros.
 * rows[] lists the n_sel row indices wanted; out is [n_sel, V] doubles.
 */
void oracle_grad_rows(const void *student, const void *teacher, int dtype,
                      int64_t V, int64_t row_stride, const int32_t *tokens,
                      const float *behav_logprob, const uint8_t *mask,
                      const int32_t *sample_id, int32_t B, const double *coef,
                      double lambda, const int64_t *rows, int64_t n_sel,
                      double *out) {
    size_t esz = dtype == ORACLE_BF16 ? 2 : 4;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t k = 0; k < n_sel; ++k) {
        int64_t n = rows[k];
        double *g = out + (size_t)k * V;
        int ok = mask[n] != 0 && tokens[n] >= 0 && tokens[n] < V &&
                 sample_id[n] >= 0 && sample_id[n] < B;
        double c = ok ? coef[sample_id[n]] : 0.0;
        if (c == 0.0) {
            for (int64_t v = 0; v < V; ++v) g[v] = 0.0;
            continue;
        }
        const void *srow = (const char *)student + (size_t)n * row_stride * esz;
        const void *trow = (const char *)teacher + (size_t)n * row_stride * esz;
        double ls = row_logsumexp(srow, dtype, V);
        double lt = row_logsumexp(trow, dtype, V);
        double kln = 0.0;
        for (int64_t v = 0; v < V; ++v) {
            double logp = logit_at(srow, dtype, v) - ls;
            double logq = logit_at(trow, dtype, v) - lt;
            kln += exp(logp) * (logp - logq);
        }
        double dn = (logit_at(srow, dtype, tokens[n]) - ls) - (double)behav_logprob[n];
        double rho_d = exp(dn) * dn;
        for (int64_t v = 0; v < V; ++v) {
            double logp = logit_at(srow, dtype, v) - ls;
            double logq = logit_at(trow, dtype, v) - lt;
            double p = exp(logp);
            double onehot = (v == tokens[n]) ? 1.0 : 0.0;
            g[v] = c * (p * ((logp - logq) - kln) + lambda * rho_d * (onehot - p));
        }
    }
}

/*
 * Sampled-token form of the token loss of Eq. 12 (Sec. 5, experimental setup;
 * Appendix B, sampled-token objectives): for an aligned row n with stored token
 * y_n ~ pi^r and rho_n = pi^t(y_n) / pi^r(y_n),
 *
 *   l_n = rho_n ( log p_s(y_n) - log p_t(y_n) )
 *
 * whose expectation over y ~ pi^r is sum_y p_s(y) (log p_s(y) - log p_t(y)).
 * out[n] = l_n for aligned rows, 0 otherwise.  lp_s, lp_t, rho, valid are the
 * arrays oracle_token_stats wrote.
 */
void oracle_sampled_token_loss(int64_t n_rows, const double *lp_s, const double *lp_t,
                               const double *rho, const uint8_t *valid, double *out) {
    for (int64_t n = 0; n < n_rows; ++n)
        out[n] = valid[n] ? rho[n] * (lp_s[n] - lp_t[n]) : 0.0;
}

/*
 * Gradient with respect to the student logits of selected rows for the
 * sampled-token loss, with w_i and the log-ratio r_n = log p_s(y_n) - log p_t(y_n)
 * held constant and the importance ratio rho_n = exp(log p_s(y_n) - b_n)
 * differentiated (d rho_n / dS_v = rho_n (1[v = y_n] - p_s(v))); the rollout
 * anchor lambda * k3(rho_n) as in oracle_grad_rows.  For c = coef_i:
 *
 *   dS[n, v] = c ( rho_n r_n + lambda rho_n d_n ) ( 1[v = y_n] - p_s(v) )
 *
 * Rows that are not aligned, or whose sample has coef = 0, get zeros.
 */
void oracle_grad_rows_sampled(const void *student, const void *teacher, int dtype,
                              int64_t V, int64_t row_stride, const int32_t *tokens,
                              const float *behav_logprob, const uint8_t *mask,
                              const int32_t *sample_id, int32_t B, const double *coef,
                              double lambda, const int64_t *rows, int64_t n_sel,
                              double *out) {
    size_t esz = dtype == ORACLE_BF16 ? 2 : 4;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t k = 0; k < n_sel; ++k) {
        int64_t n = rows[k];
        double *g = out + (size_t)k * V;
        int ok = mask[n] != 0 && tokens[n] >= 0 && tokens[n] < V &&
                 sample_id[n] >= 0 && sample_id[n] < B;
        double c = ok ? coef[sample_id[n]] : 0.0;
        if (c == 0.0) {
            for (int64_t v = 0; v < V; ++v) g[v] = 0.0;
            continue;
        }
        const void *srow = (const char *)student + (size_t)n * row_stride * esz;
        const void *trow = (const char *)teacher + (size_t)n * row_stride * esz;
        double ls = row_logsumexp(srow, dtype, V);
        double lt = row_logsumexp(trow, dtype, V);
        double lps = logit_at(srow, dtype, tokens[n]) - ls;
        double lpt = logit_at(trow, dtype, tokens[n]) - lt;
        double dn = lps - (double)behav_logprob[n];
        double rho = exp(dn);
        double weight = c * (rho * (lps - lpt) + lambda * rho * dn);
        for (int64_t v = 0; v < V; ++v) {
            double p = exp(logit_at(srow, dtype, v) - ls);
            double onehot = (v == tokens[n]) ? 1.0 : 0.0;
            g[v] = weight * (onehot - p);
        }
    }
}
