/*
 * bebop_oracle.c -- plain, slow, fp64 CPU statement of the speculative
 * rejection-sampling verify step.  TEST INFRASTRUCTURE ONLY: nothing on the
 * product path may include, link or call this file; it shares no code with
 * the CUDA kernels.
 *
 * What each function follows (paper = "Breaking Entropy Bounds: Accelerating
 * RL Training via MTP with Rejection Sampling"):
 *   softmax with temperature ............ Sec. 2.2, App. G.1 "Draft stage"
 *   total variation, three equal forms .. Eq. (reject_sample), Sec. 3.3 identity
 *   accept scan, residual, inverse CDF .. Algorithm 3 (App. G.1), in its order
 *   greedy (argmax-match) mode .......... deterministic limit of Sec. 2.2 "Target-Only"
 *
 * Readings taken where the paper is silent or inconsistent:
 *   - bonus token: drawn from the target row AFTER the last draft (row L of
 *     the K+1 target rows), so that every emitted position is distributed as p.
 *   - accept iff u*q(x) < p(x) (strict), product form, no division.
 *   - inverse CDF: smallest v with C(v) >= u*Z (Algorithm 3's ">=").
 *   - Z == 0 at a rejected position: draw from p of that position, status bit 8.
 *   - ragged rows: tv = p_draft = q_draft = 0 and tokens = -1 past draft_len.
 *   - argmax ties: lowest index.
 *   Parity unpinned (pure conventions, nothing in the paper fixes them):
 *   the Z == 0 fallback, ragged padding values, the status-bit values.
 *
 * Sums run left to right in long double (x87 80-bit on x86-64) so that the
 * oracle's own rounding is far below every margin it reports.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ST_NONFINITE 1   /* NaN or +inf logit in a row the method reads      */
#define ST_EMPTY_ROW 2   /* a row whose logits are all -inf                  */
#define ST_BAD_TOKEN 4   /* draft token id outside [0, V)                    */
#define ST_ZERO_RESID 8  /* residual mass 0 at a rejected position           */
#define ST_BAD_TEMP 16   /* temperature <= 0 or non-finite                   */
#define ST_FATAL (ST_NONFINITE | ST_EMPTY_ROW | ST_BAD_TOKEN | ST_BAD_TEMP)

/* softmax(z / tau) over the full vocabulary, max-subtracted, in double.
 * Returns status bits (0, ST_NONFINITE, ST_EMPTY_ROW). -inf logits are legal
 * and get probability exactly 0. */
int oracle_softmax(const float *z, int64_t V, double tau, double *prob)
{
    double m = -INFINITY;
    for (int64_t v = 0; v < V; ++v) {
        double x = (double)z[v] / tau;
        if (isnan(x) || x == INFINITY) return ST_NONFINITE;
        if (x > m) m = x;
    }
    if (m == -INFINITY) return ST_EMPTY_ROW;
    long double S = 0.0L;
    for (int64_t v = 0; v < V; ++v) {
        double x = (double)z[v] / tau;
        prob[v] = (x == -INFINITY) ? 0.0 : exp(x - m);
        S += prob[v];
    }
    for (int64_t v = 0; v < V; ++v) prob[v] = (double)((long double)prob[v] / S);
    return 0;
}

/* The three equal expressions of d_TV(p,q):
 *   out[0] = sum_v max(0, p-q)      (the residual mass Z of Algorithm 3)
 *   out[1] = 1 - sum_v min(p,q)     (Eq. reject_sample / Sec. 3.3)
 *   out[2] = 1/2 sum_v |p-q|        (definition)                             */
void oracle_tv3(const double *p, const double *q, int64_t V, double out[3])
{
    long double a = 0.0L, b = 0.0L, c = 0.0L;
    for (int64_t v = 0; v < V; ++v) {
        double d = p[v] - q[v];
        a += (d > 0.0) ? d : 0.0;
        b += (p[v] < q[v]) ? p[v] : q[v];
        c += fabs(d);
    }
    out[0] = (double)a;
    out[1] = (double)(1.0L - b);
    out[2] = (double)(0.5L * c);
}

static double clamp01(double x) { return x < 0.0 ? 0.0 : (x > 1.0 ? 1.0 : x); }

/* Inverse CDF over r[0..V): smallest v with C(v) >= u*Z, Z = C(V-1).
 * Also reports how far t = u*Z lies from the edges of the selected token's
 * CDF interval, relative to that token's mass (margin_tok) and relative to t
 * (margin_t). */
static int64_t inverse_cdf(const double *r, int64_t V, double u, double *Z_out,
                           double *margin_tok, double *margin_t)
{
    long double Z = 0.0L;
    for (int64_t v = 0; v < V; ++v) Z += r[v];
    *Z_out = (double)Z;
    long double t = (long double)u * Z;
    long double C = 0.0L, Cprev = 0.0L;
    int64_t y = -1;
    for (int64_t v = 0; v < V; ++v) {
        Cprev = C;
        C += r[v];
        if (C >= t) { y = v; break; }
    }
    if (y < 0) { /* cannot happen: C(V-1) == Z >= u*Z for u < 1 */
        for (int64_t v = V - 1; v >= 0; --v) if (r[v] > 0.0) { y = v; break; }
        *margin_tok = 0.0; *margin_t = 0.0;
        return y;
    }
    long double lo = t - Cprev, hi = C - t;
    long double gap = lo < hi ? lo : hi;
    *margin_tok = (r[y] > 0.0) ? (double)(gap / (long double)r[y]) : 0.0;
    *margin_t = (t > 0.0L) ? (double)(gap / t) : 0.0;
    return y;
}

static void verify_one(const float *target, int64_t ld_t, const float *draft, int64_t ld_d,
                       const int32_t *tok, int L, double tau, const float *u_acc, double u_fin,
                       int K, int64_t V,
                       int32_t *accept_len, int32_t *out_tokens, double *tv, double *p_draft,
                       double *q_draft, int32_t *status, double *margin_acc, double *margin_cdf,
                       double *margin_cdf_t, double *p, double *q, double *r)
{
    int st = 0;
    double Z;
    int64_t y;
    *accept_len = 0;
    for (int k = 0; k <= K; ++k) out_tokens[k] = -1;
    for (int k = 0; k < K; ++k) { tv[k] = 0.0; p_draft[k] = 0.0; q_draft[k] = 0.0; margin_acc[k] = INFINITY; }
    *margin_cdf = INFINITY; *margin_cdf_t = INFINITY;

    if (!(tau > 0.0) || !isfinite(tau)) { *status = ST_BAD_TEMP; return; }
    for (int k = 0; k < L; ++k) if (tok[k] < 0 || tok[k] >= V) st |= ST_BAD_TOKEN;
    if (st) { *status = st; return; }

    /* Steps 1-3: every draft position gets its softmax pair, its TV and the
     * gathered probabilities; the accept scan stops at the first reject. */
    int n = L, stopped = 0;
    for (int k = 0; k < L; ++k) {
        st |= oracle_softmax(target + (int64_t)k * ld_t, V, tau, p);
        st |= oracle_softmax(draft + (int64_t)k * ld_d, V, tau, q);
        if (st & ST_FATAL) break;
        double t3[3];
        oracle_tv3(p, q, V, t3);
        tv[k] = clamp01(t3[0]);
        double px = p[tok[k]], qx = q[tok[k]];
        p_draft[k] = px; q_draft[k] = qx;
        if (!stopped) {
            double lhs = (double)u_acc[k] * qx;          /* u_k * q_k(x_k) */
            double big = lhs > px ? lhs : px;
            margin_acc[k] = big > 0.0 ? fabs(lhs - px) / big : 0.0;
            if (lhs >= px) {                              /* reject */
                n = k; stopped = 1;
                for (int64_t v = 0; v < V; ++v) { double d = p[v] - q[v]; r[v] = d > 0.0 ? d : 0.0; }
            }
        }
    }
    if (st & ST_FATAL) goto fatal;

    /* Steps 4-5: residual at the rejected position, or the bonus row. */
    if (!stopped) {
        st |= oracle_softmax(target + (int64_t)L * ld_t, V, tau, p);
        if (st & ST_FATAL) goto fatal;
        y = inverse_cdf(p, V, u_fin, &Z, margin_cdf, margin_cdf_t);
    } else {
        y = inverse_cdf(r, V, u_fin, &Z, margin_cdf, margin_cdf_t);
        if (!(Z > 0.0)) {                                 /* reading for Z == 0 */
            st |= ST_ZERO_RESID;
            oracle_softmax(target + (int64_t)n * ld_t, V, tau, p);
            y = inverse_cdf(p, V, u_fin, &Z, margin_cdf, margin_cdf_t);
        }
    }
    *accept_len = n;
    for (int k = 0; k < n; ++k) out_tokens[k] = tok[k];
    out_tokens[n] = (int32_t)y;
    *status = st;
    return;

fatal:
    *accept_len = 0;
    for (int k = 0; k < K; ++k) { tv[k] = 0.0; p_draft[k] = 0.0; q_draft[k] = 0.0; margin_acc[k] = INFINITY; }
    *status = st;
}

/* Chain rejection-sampling verification for B sequences (Algorithm 3 per
 * sequence).  All pointers are host pointers.
 *   target [B, K+1, ld_t], draft [B, K, ld_d] (floats; bf16 inputs are widened
 *   exactly by the caller), draft_tokens [B,K], draft_len [B] or NULL (= K),
 *   temperature [B] or NULL (= temperature_all), u_accept [B,K], u_final [B].
 * Outputs: accept_len [B], out_tokens [B,K+1], tv/p_draft/q_draft [B,K]
 * (double), row_status [B], margin_acc [B,K] (+inf where the test was not
 * evaluated), margin_cdf [B] (relative to the chosen token's mass),
 * margin_cdf_t [B] (relative to u*Z).  Returns 0, or -1 on allocation failure. */
int oracle_verify(const float *target, int64_t ld_t, const float *draft, int64_t ld_d,
                  const int32_t *draft_tokens, const int32_t *draft_len,
                  const float *temperature, float temperature_all,
                  const float *u_accept, const float *u_final,
                  int B, int K, int64_t V,
                  int32_t *accept_len, int32_t *out_tokens, double *tv, double *p_draft,
                  double *q_draft, int32_t *row_status, double *margin_acc,
                  double *margin_cdf, double *margin_cdf_t, int nthreads)
{
    int fail = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#pragma omp parallel
#endif
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)V);
        double *q = (double *)malloc(sizeof(double) * (size_t)V);
        double *r = (double *)malloc(sizeof(double) * (size_t)V);
        if (!p || !q || !r) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            fail = 1;
        } else {
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
            for (int b = 0; b < B; ++b) {
                int L = draft_len ? draft_len[b] : K;
                if (L < 0) L = 0;
                if (L > K) L = K;
                double tau = temperature ? (double)temperature[b] : (double)temperature_all;
                verify_one(target + (int64_t)b * (K + 1) * ld_t, ld_t,
                           draft + (int64_t)b * K * ld_d, ld_d,
                           draft_tokens + (int64_t)b * K, L, tau,
                           u_accept + (int64_t)b * K, (double)u_final[b], K, V,
                           accept_len + b, out_tokens + (int64_t)b * (K + 1),
                           tv + (int64_t)b * K, p_draft + (int64_t)b * K, q_draft + (int64_t)b * K,
                           row_status + b, margin_acc + (int64_t)b * K, margin_cdf + b,
                           margin_cdf_t + b, p, q, r);
            }
        }
        free(p); free(q); free(r);
    }
    return fail ? -1 : 0;
}

/* TV of N independent row pairs: tv[n] = sum_v max(0, p-q) clamped to [0,1],
 * s_aux[n] = sum_v q(v) * 1[q(v) <= p(v)] (the scalar S of Eq. tv_grad /
 * Algorithm 1), row_status[n] as above.  tv3 (may be NULL) receives the three
 * unclamped forms, [N,3]. */
int oracle_tv(const float *target, int64_t ld_t, const float *draft, int64_t ld_d,
              const float *temperature, float temperature_all, int N, int64_t V,
              double *tv, double *s_aux, int32_t *row_status, double *tv3, int nthreads)
{
    int fail = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#pragma omp parallel
#endif
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)V);
        double *q = (double *)malloc(sizeof(double) * (size_t)V);
        if (!p || !q) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            fail = 1;
        } else {
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
            for (int n = 0; n < N; ++n) {
                double tau = temperature ? (double)temperature[n] : (double)temperature_all;
                int st = 0;
                tv[n] = 0.0; s_aux[n] = 0.0;
                if (tv3) { tv3[3 * n] = tv3[3 * n + 1] = tv3[3 * n + 2] = 0.0; }
                if (!(tau > 0.0) || !isfinite(tau)) { row_status[n] = ST_BAD_TEMP; continue; }
                st |= oracle_softmax(target + (int64_t)n * ld_t, V, tau, p);
                st |= oracle_softmax(draft + (int64_t)n * ld_d, V, tau, q);
                row_status[n] = st;
                if (st & ST_FATAL) continue;
                double t3[3];
                oracle_tv3(p, q, V, t3);
                tv[n] = clamp01(t3[0]);
                if (tv3) { tv3[3 * n] = t3[0]; tv3[3 * n + 1] = t3[1]; tv3[3 * n + 2] = t3[2]; }
                long double S = 0.0L;
                for (int64_t v = 0; v < V; ++v) if (q[v] <= p[v]) S += q[v];
                s_aux[n] = (double)S;
            }
        }
        free(p); free(q);
    }
    return fail ? -1 : 0;
}

/* Greedy-draft mode: g_k = lowest index attaining max_v target[b,k,v];
 * accept while x_k == g_k; emit g at the stop position (g_L when all L are
 * accepted).  Temperature plays no role.  All L+1 target rows are examined.  */
int oracle_greedy_verify(const float *target, int64_t ld_t, const int32_t *draft_tokens,
                         const int32_t *draft_len, int B, int K, int64_t V,
                         int32_t *accept_len, int32_t *out_tokens, int32_t *row_status,
                         int nthreads)
{
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int b = 0; b < B; ++b) {
        int L = draft_len ? draft_len[b] : K;
        if (L < 0) L = 0;
        if (L > K) L = K;
        const int32_t *tok = draft_tokens + (int64_t)b * K;
        int32_t *out = out_tokens + (int64_t)b * (K + 1);
        int st = 0;
        for (int k = 0; k <= K; ++k) out[k] = -1;
        accept_len[b] = 0;
        for (int k = 0; k < L; ++k) if (tok[k] < 0 || tok[k] >= V) st |= ST_BAD_TOKEN;
        int64_t g[64];
        for (int k = 0; k <= L && k < 64; ++k) {
            const float *z = target + ((int64_t)b * (K + 1) + k) * ld_t;
            float m = -INFINITY; int64_t arg = -1;
            for (int64_t v = 0; v < V; ++v) {
                if (isnan(z[v]) || z[v] == INFINITY) st |= ST_NONFINITE;
                if (z[v] > m) { m = z[v]; arg = v; }
            }
            if (arg < 0) st |= ST_EMPTY_ROW;
            g[k] = arg;
        }
        row_status[b] = st;
        if (st & ST_FATAL) continue;
        int n = 0;
        while (n < L && tok[n] == g[n]) ++n;
        accept_len[b] = n;
        for (int k = 0; k < n; ++k) out[k] = tok[k];
        out[n] = (int32_t)g[n];
    }
    return 0;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
