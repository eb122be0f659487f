/*
 * sgbv_oracle.c -- float64 CPU oracle for multi-draft greedy block verification (SpecTr-GBV).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the paper's
 * verification step computes (Algorithm 1 with Eqs. 2, 3 and 4).  Only the test-suite, the
 * smoke check and the CPU-baseline leg of the benchmark may call it.  It shares no code,
 * header, table or helper with the CUDA path and must never be reached from the product path.
 *
 * Notation (0-based tensors, paper symbols in brackets):
 *   B, K, gamma [L], V [|Omega|]        batch rows, drafts per row, draft length, vocabulary
 *   zq[b,k,i,:]  i = 0..gamma           target logits after the first i tokens of draft k
 *   zp[b,k,i,:]  i = 0..gamma-1         draft  logits after the same prefix
 *   tok[b,k,i]   i = 0..gamma-1         draft token x_k^{(i+1)}
 *   q_i, p_i                            softmax(z/T) of those rows        (Preliminaries)
 *   a_i = q(x_k^i), b_i = p(x_k^i)      joint prefix probabilities, a_0 = b_0 = 1
 *   S_i = sum_x q(x^i,x) (1 - min{p(x^i,x)/q(x^i,x), 1})^K        (sum of Eqs. 2 and 4)
 *   h[k][i-1], i = 1..gamma             acceptance weight of the length-i sub-block (Eqs. 2, 3)
 *   uniforms[b, k*gamma + (i-1)]        eta of the trial on sub-block (k,i);  last entry: u_s
 *
 * Readings taken where the paper is silent (each is also a comment at the place it applies):
 *   - the test "eta < h" is strict; eta is pre-drawn per (k,i) and consumed whether used or not;
 *   - H holds rejected/skipped sub-blocks; membership = equal length and equal tokens;
 *   - the whole-block accept also records f = k;
 *   - tau = 0 uses the rows of draft 0 at position 0 with a = b = 1, and reports f = -1;
 *   - h is clamped to [0,1]; Eq. 2 with a vanishing denominator (0/0) gives h = 1, as
 *     single-draft GBV does at K = 1; Eq. 3 with a vanishing denominator gives h = 0;
 *   - a residual with zero total mass falls back to q of the same row (flagged);
 *   - inverse CDF: ascending vocabulary index, first x with cumulative mass > u_s * total;
 *     if rounding leaves none, the last x with positive mass;
 *   - one temperature T > 0 divides the logits of both models.
 *
 * Also here, with their own pins: one position of Algorithm 2 (sgbv_oracle_modify) and the comparison
 * verifiers of Section 3, token-level speculative sampling and SpecTr's K-SEQ (sgbv_oracle_kseq_verify).
 *
 * Pins (tests, CPU only): the K=1 case against an independent single-draft GBV; K=1,gamma=1
 * against token-level speculative sampling; exactness of the output law at K=1 by exhaustive
 * enumeration on tree models; the hand-derived two-token example (19/27); closed forms of S on
 * special rows; the algebraic identity behind Eq. 2 (Lemma A.1); Monte-Carlo against the
 * enumerated law.  The "gamma = 1 equals SpecTr's K-SEQ" statement is NOT asserted: at
 * gamma = 1 the method solves the same per-position problem with a different rule, so
 * numerical parity with K-SEQ is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_STATUS_TOKEN_RANGE 1
#define ORACLE_STATUS_NONFINITE 2
#define ORACLE_STATUS_DEGENERATE_RESIDUAL 4

/* ---- step 1: temperature softmax of one vocabulary row ------------------------------------ */
/* q(x) = exp(z_x/T) / sum_x' exp(z_x'/T), evaluated with the row maximum subtracted.
 * Returns log sum_x exp(z_x/T) (the log-normaliser).  prob may be NULL. */
double sgbv_oracle_softmax(const float *z, int V, double T, double *prob) {
    double m = -INFINITY;
    for (int x = 0; x < V; ++x) {
        double s = (double)z[x] / T;
        if (s > m) m = s;
    }
    double Z = 0.0;
    for (int x = 0; x < V; ++x) Z += exp((double)z[x] / T - m);
    if (prob) {
        for (int x = 0; x < V; ++x) prob[x] = exp((double)z[x] / T - m) / Z;
    }
    return m + log(Z);
}

/* g(u) = 1 - (1-u)^K, the probability that at least one of K i.i.d. drafts hits an event of
 * probability u (Lemma A.1's marginal).  Evaluated as -expm1(K log1p(-u)) so that tiny u does
 * not round to 0; the function is the same. */
double sgbv_oracle_g(double u, int K) {
    if (u >= 1.0) return 1.0;
    if (u <= 0.0) return 0.0;
    return -expm1((double)K * log1p(-u));
}

/* ---- step 3: un-normalised residual mass --------------------------------------------------- */
/* S = sum_x q(x^i,x) (1 - min{p(x^i,x)/q(x^i,x), 1})^K with q(x^i,x) = a q(x), p(x^i,x) = b p(x)
 * (first sum of Eq. 2 = denominator of Eq. 4).  Terms with q(x^i,x) = 0 contribute 0.
 * If w != NULL it receives the V summands (the un-normalised Eq. 4). */
double sgbv_oracle_resmass(const double *q, const double *p, int V, double a, double b, int K,
                           double *w) {
    double S = 0.0;
    for (int x = 0; x < V; ++x) {
        double qj = a * q[x];
        double pj = b * p[x];
        double term = 0.0;
        if (qj > 0.0) {
            double r = pj / qj;
            if (r > 1.0) r = 1.0;
            term = qj * pow(1.0 - r, (double)K);
        }
        if (w) w[x] = term;
        S += term;
    }
    return S;
}

static double clamp01(double x) {
    if (!(x > 0.0)) return 0.0;
    return x > 1.0 ? 1.0 : x;
}

/* ---- step 4: acceptance weights ------------------------------------------------------------- */
/* Eq. 2: weight of a proper sub-block of length i (1 <= i <= gamma-1); a = q(x^i), b = p(x^i),
 * S = residual mass of the row that follows the sub-block.
 * Reading for 0/0: numerator <= denominator always (g is concave), and the denominator
 * vanishes exactly when every draft continuation of x^i is accepted anyway (at K = 1: when
 * b p(x) <= a q(x) for all x, where single-draft GBV's ratio is +inf, i.e. "accept").  So a
 * denominator at the rounding floor of its own terms gives h = 1. */
double sgbv_oracle_h_sub(double a, double b, double S, int K) {
    double r = (a > 0.0) ? b / a : 1.0;
    if (r > 1.0) r = 1.0;
    double gb = sgbv_oracle_g(b, K);
    double num = S - a * pow(1.0 - r, (double)K);
    double den = gb - a + S;
    if (!(den > 1e-12 * (gb + a))) return 1.0;
    return clamp01(num / den);
}

/* Eq. 3: weight of the whole block; a = q(x^L), b = p(x^L).  A block of zero draft probability
 * (denominator 0) gets weight 0. */
double sgbv_oracle_h_full(double a, double b, int K) {
    double r = (a > 0.0) ? b / a : 1.0;
    if (r > 1.0) r = 1.0;
    double num = a * sgbv_oracle_g(r, K);
    double den = sgbv_oracle_g(b, K);
    if (!(den > 0.0)) return 0.0;
    return clamp01(num / den);
}

/* ---- step 5: the scan of Algorithm 1 -------------------------------------------------------- */
static int in_H(const int32_t *H_tok, const int *H_len, int nH, int gamma, const int32_t *blk,
                int len) {
    for (int j = 0; j < nH; ++j) {
        if (H_len[j] != len) continue;
        if (memcmp(H_tok + (size_t)j * gamma, blk, (size_t)len * sizeof(int32_t)) == 0) return 1;
    }
    return 0;
}

/* h[k*gamma + (i-1)], tok[k*gamma + i], eta[k*gamma + (i-1)].  Writes tau (0..gamma) and the
 * accepted draft f (-1 when tau = 0). */
void sgbv_oracle_scan(const double *h, const int32_t *tok, const float *eta, int K, int gamma,
                      int32_t *out_tau, int32_t *out_f) {
    int tau = 0, f = -1, nH = 0;
    int32_t *H_tok = (int32_t *)malloc((size_t)K * gamma * gamma * sizeof(int32_t));
    int *H_len = (int *)malloc((size_t)K * gamma * sizeof(int));
    int done = 0;
    for (int k = 0; k < K && !done; ++k) {
        const int32_t *blk = tok + (size_t)k * gamma;
        int start = tau + 1; /* loop bounds are fixed when the draft is entered */
        for (int i = start; i <= gamma; ++i) {
            double hv = h[(size_t)k * gamma + (i - 1)];
            double e = (double)eta[(size_t)k * gamma + (i - 1)];
            int accept = (e < hv) && !in_H(H_tok, H_len, nH, gamma, blk, i);
            if (accept) {
                tau = i; /* the sub-block of draft k replaces the accepted block wholesale */
                f = k;
                if (i == gamma) { /* whole block accepted: stop all loops */
                    done = 1;
                    break;
                }
            } else {
                memcpy(H_tok + (size_t)nH * gamma, blk, (size_t)i * sizeof(int32_t));
                H_len[nH] = i;
                ++nH;
            }
        }
    }
    free(H_tok);
    free(H_len);
    *out_tau = tau;
    *out_f = f;
}

/* ---- step 6: inverse-CDF sample -------------------------------------------------------------- */
/* y = min{x : sum_{x'<=x} w_x' > u * sum w}.  margin (may be NULL) receives the distance of u to
 * the nearer normalised CDF edge of the chosen cell.  Returns -1 if the total mass is 0. */
int32_t sgbv_oracle_sample(const double *w, int V, double u, double *margin) {
    double W = 0.0;
    for (int x = 0; x < V; ++x) W += w[x];
    if (!(W > 0.0)) return -1;
    double target = u * W, cum = 0.0;
    int32_t last_pos = -1;
    for (int x = 0; x < V; ++x) {
        double prev = cum;
        cum += w[x];
        if (w[x] > 0.0) last_pos = x;
        if (cum > target) {
            if (margin) {
                double lo = fabs(u - prev / W), hi = fabs(cum / W - u);
                *margin = lo < hi ? lo : hi;
            }
            return x;
        }
    }
    if (margin) *margin = 0.0;
    return last_pos;
}

/* ---- whole verify step for one batch row ------------------------------------------------------ */
static void verify_row(const float *zq, const float *zp, const int32_t *tok, const float *u, int K,
                       int gamma, int V, double T, int32_t *out_tau, int32_t *out_f,
                       int32_t *out_tokens, double *out_h, double *out_S, double *out_loga,
                       double *out_logb, int32_t *out_status, double *out_margin_accept,
                       double *out_margin_sample) {
    int status = 0;
    double *q = (double *)malloc((size_t)V * sizeof(double));
    double *p = (double *)malloc((size_t)V * sizeof(double));
    double *h = (double *)malloc((size_t)K * gamma * sizeof(double));
    double *S = (double *)malloc((size_t)K * gamma * sizeof(double));
    double *la = (double *)malloc((size_t)K * (gamma + 1) * sizeof(double));
    double *lb = (double *)malloc((size_t)K * (gamma + 1) * sizeof(double));
    double *av = (double *)malloc((size_t)K * (gamma + 1) * sizeof(double)); /* a_i = q(x_k^i) */
    double *bv = (double *)malloc((size_t)K * (gamma + 1) * sizeof(double)); /* b_i = p(x_k^i) */

    /* rows the method reads up front: target rows i < gamma and every draft row.  A NaN or +inf
     * logit, or a row without any finite logit, invalidates the batch row.  (The target row
     * i = gamma of a draft is read only after a full accept and is checked there.) */
    for (int k = 0; k < K; ++k)
        for (int i = 0; i < gamma; ++i) {
            const float *rq = zq + ((size_t)k * (gamma + 1) + i) * V;
            const float *rp = zp + ((size_t)k * gamma + i) * V;
            int anyq = 0, anyp = 0;
            for (int x = 0; x < V; ++x) {
                if (isnan(rq[x]) || rq[x] == INFINITY || isnan(rp[x]) || rp[x] == INFINITY)
                    status |= ORACLE_STATUS_NONFINITE;
                anyq |= isfinite(rq[x]);
                anyp |= isfinite(rp[x]);
            }
            if (!anyq || !anyp) status |= ORACLE_STATUS_NONFINITE;
        }
    for (int n = 0; n < K * gamma; ++n)
        if (tok[n] < 0 || tok[n] >= V) status |= ORACLE_STATUS_TOKEN_RANGE;

    if (status == 0) {
        for (int k = 0; k < K; ++k) {
            double a = 1.0, b = 1.0; /* a_0 = b_0 = 1 */
            double loga = 0.0, logb = 0.0;
            for (int i = 0; i < gamma; ++i) {
                const float *zq_row = zq + ((size_t)k * (gamma + 1) + i) * V;
                const float *zp_row = zp + ((size_t)k * gamma + i) * V;
                double lse_q = sgbv_oracle_softmax(zq_row, V, T, q);
                double lse_p = sgbv_oracle_softmax(zp_row, V, T, p);
                la[k * (gamma + 1) + i] = loga;
                lb[k * (gamma + 1) + i] = logb;
                av[k * (gamma + 1) + i] = a;
                bv[k * (gamma + 1) + i] = b;
                /* S_i with the joint probabilities of the length-i prefix of draft k */
                S[k * gamma + i] = sgbv_oracle_resmass(q, p, V, a, b, K, NULL);
                if (i >= 1) h[k * gamma + (i - 1)] = sgbv_oracle_h_sub(a, b, S[k * gamma + i], K);
                int32_t t = tok[k * gamma + i];
                a *= q[t]; /* a_{i+1} = a_i q_i(tok_i) */
                b *= p[t];
                loga += (double)zq_row[t] / T - lse_q;
                logb += (double)zp_row[t] / T - lse_p;
            }
            la[k * (gamma + 1) + gamma] = loga;
            lb[k * (gamma + 1) + gamma] = logb;
            av[k * (gamma + 1) + gamma] = a;
            bv[k * (gamma + 1) + gamma] = b;
            h[k * gamma + (gamma - 1)] = sgbv_oracle_h_full(a, b, K);
        }

        int32_t tau, f;
        sgbv_oracle_scan(h, tok, u, K, gamma, &tau, &f);

        double margin_a = INFINITY;
        for (int n = 0; n < K * gamma; ++n) {
            double d = fabs((double)u[n] - h[n]);
            if (d < margin_a) margin_a = d;
        }

        /* extra token: residual of Eq. 4 after the accepted block, or the bonus draw from q */
        int kk = (tau == 0) ? 0 : f;
        double us = (double)u[K * gamma];
        double margin_s = 0.0;
        int32_t y;
        const float *zq_row = zq + ((size_t)kk * (gamma + 1) + tau) * V;
        sgbv_oracle_softmax(zq_row, V, T, q);
        if (tau < gamma) {
            const float *zp_row = zp + ((size_t)kk * gamma + tau) * V;
            sgbv_oracle_softmax(zp_row, V, T, p);
            /* joint probabilities of the accepted block; a_0 = b_0 = 1 when tau = 0 */
            double a = av[kk * (gamma + 1) + tau], b = bv[kk * (gamma + 1) + tau];
            double *w = (double *)malloc((size_t)V * sizeof(double));
            sgbv_oracle_resmass(q, p, V, a, b, K, w);
            y = sgbv_oracle_sample(w, V, us, &margin_s);
            free(w);
            if (y < 0) { /* zero residual mass: fall back to q of the same row */
                status |= ORACLE_STATUS_DEGENERATE_RESIDUAL;
                y = sgbv_oracle_sample(q, V, us, &margin_s);
            }
        } else {
            int any = 0, badrow = 0; /* bonus row: checked when it is actually read */
            for (int x = 0; x < V; ++x) {
                badrow |= isnan(zq_row[x]) || zq_row[x] == INFINITY;
                any |= isfinite(zq_row[x]);
            }
            if (badrow || !any) {
                status |= ORACLE_STATUS_NONFINITE;
                y = -1;
            } else {
                y = sgbv_oracle_sample(q, V, us, &margin_s);
            }
        }

        for (int i = 0; i <= gamma; ++i) out_tokens[i] = -1;
        if (status & ORACLE_STATUS_NONFINITE) {
            tau = -1;
            f = -1;
        } else {
            for (int i = 0; i < tau; ++i) out_tokens[i] = tok[f * gamma + i];
            out_tokens[tau] = y;
        }
        *out_tau = tau;
        *out_f = f;
        if (out_margin_accept) *out_margin_accept = margin_a;
        if (out_margin_sample) *out_margin_sample = margin_s;
        if (out_h) memcpy(out_h, h, (size_t)K * gamma * sizeof(double));
        if (out_S) memcpy(out_S, S, (size_t)K * gamma * sizeof(double));
        if (out_loga) memcpy(out_loga, la, (size_t)K * (gamma + 1) * sizeof(double));
        if (out_logb) memcpy(out_logb, lb, (size_t)K * (gamma + 1) * sizeof(double));
    } else {
        *out_tau = -1;
        *out_f = -1;
        for (int i = 0; i <= gamma; ++i) out_tokens[i] = -1;
        if (out_margin_accept) *out_margin_accept = 0.0;
        if (out_margin_sample) *out_margin_sample = 0.0;
        if (out_h) for (int n = 0; n < K * gamma; ++n) out_h[n] = NAN;
        if (out_S) for (int n = 0; n < K * gamma; ++n) out_S[n] = NAN;
        if (out_loga) for (int n = 0; n < K * (gamma + 1); ++n) out_loga[n] = NAN;
        if (out_logb) for (int n = 0; n < K * (gamma + 1); ++n) out_logb[n] = NAN;
    }
    if (out_status) *out_status = status;
    free(q); free(p); free(h); free(S); free(la); free(lb); free(av); free(bv);
}

/* Whole batch.  All pointers are host pointers.  Diagnostic outputs may be NULL.
 *   zq [B,K,gamma+1,V]  zp [B,K,gamma,V]  tok [B,K,gamma]  uniforms [B,K*gamma+1]
 *   out_tau [B]  out_f [B]  out_tokens [B,gamma+1]
 *   out_h [B,K,gamma]  out_S [B,K,gamma]  out_loga/out_logb [B,K,gamma+1]
 *   out_status [B]  out_margin_accept [B]  out_margin_sample [B]
 * nthreads <= 0: all cores.  Returns the number of threads used, or -1 on a bad argument. */
int sgbv_oracle_verify(const float *zq, const float *zp, const int32_t *tok, const float *uniforms,
                       int B, int K, int gamma, int V, double T, int32_t *out_tau, int32_t *out_f,
                       int32_t *out_tokens, double *out_h, double *out_S, double *out_loga,
                       double *out_logb, int32_t *out_status, double *out_margin_accept,
                       double *out_margin_sample, int nthreads) {
    if (B < 0 || K < 1 || gamma < 1 || V < 1 || !(T > 0.0) || !isfinite(T)) return -1;
    int used = 1;
#ifdef _OPENMP
    if (nthreads <= 0) nthreads = omp_get_max_threads();
    if (nthreads > B && B > 0) nthreads = B;
    used = nthreads;
#pragma omp parallel for schedule(dynamic, 1) num_threads(nthreads)
#endif
    for (int b = 0; b < B; ++b) {
        verify_row(zq + (size_t)b * K * (gamma + 1) * V, zp + (size_t)b * K * gamma * V,
                   tok + (size_t)b * K * gamma, uniforms + (size_t)b * (K * gamma + 1), K, gamma, V,
                   T, out_tau + b, out_f + b, out_tokens + (size_t)b * (gamma + 1),
                   out_h ? out_h + (size_t)b * K * gamma : NULL,
                   out_S ? out_S + (size_t)b * K * gamma : NULL,
                   out_loga ? out_loga + (size_t)b * K * (gamma + 1) : NULL,
                   out_logb ? out_logb + (size_t)b * K * (gamma + 1) : NULL,
                   out_status ? out_status + b : NULL,
                   out_margin_accept ? out_margin_accept + b : NULL,
                   out_margin_sample ? out_margin_sample + b : NULL);
    }
    return used;
}

/* ============================================================================================== */
/* Algorithm 2 (Distribution Modification), one position.                                          */
/*                                                                                                 */
/* After an iteration that stopped short (tau < L), the next L - tau - 1 tokens are drawn from    */
/*   q_new(x) = q(s,x) (1 - min{p(s,x)/q(s,x), 1})^K / sum_x' q(s,x') (1 - min{p(s,x')/q(s,x'),1})^K */
/* where s = (t^tau, y, x^{i-1}) is everything emitted so far and q(s,x) = a q(x|s), p(s,x) =      */
/* b p(x|s) are JOINT probabilities, a = q(s), b = p(s) carried along as logarithms.  The common   */
/* factor a cancels between numerator and denominator, so the sums are formed with (1, b/a) in     */
/* place of (a, b): same distribution, and a long s cannot underflow it.                           */
/*   zq, zp [B,V] logits of the position; loga, logb [B]; u [B] uniforms for the inverse CDF       */
/*   out_token [B]; out_loga/out_logb [B] = carried logs with the drawn token appended;            */
/*   out_R [B] = sum_x q(x|s)(1 - min{(b/a) p(x|s)/q(x|s), 1})^K; out_qnew [B,V] or NULL;          */
/*   out_status [B]; out_margin [B] (distance of u to the nearer CDF edge of the drawn cell).      */
/* Zero total mass: the token is drawn from q(.|s) itself (flagged), as for Eq. 4.                 */
int sgbv_oracle_modify(const float *zq, const float *zp, const double *loga, const double *logb,
                       const float *u, int B, int V, int K, double T, int32_t *out_token,
                       double *out_loga, double *out_logb, double *out_R, double *out_qnew,
                       int32_t *out_status, double *out_margin) {
    if (B < 0 || V < 1 || K < 1 || !(T > 0.0) || !isfinite(T)) return -1;
    for (int b = 0; b < B; ++b) {
        const float *rq = zq + (size_t)b * V, *rp = zp + (size_t)b * V;
        int status = 0, anyq = 0, anyp = 0;
        for (int x = 0; x < V; ++x) {
            if (isnan(rq[x]) || rq[x] == INFINITY || isnan(rp[x]) || rp[x] == INFINITY)
                status |= ORACLE_STATUS_NONFINITE;
            anyq |= isfinite(rq[x]);
            anyp |= isfinite(rp[x]);
        }
        if (!anyq || !anyp) status |= ORACLE_STATUS_NONFINITE;
        int32_t y = -1;
        double R = NAN, la = NAN, lb = NAN, margin = 0.0;
        if (status == 0) {
            double *q = (double *)malloc((size_t)V * sizeof(double));
            double *p = (double *)malloc((size_t)V * sizeof(double));
            double *w = (double *)malloc((size_t)V * sizeof(double));
            double lse_q = sgbv_oracle_softmax(rq, V, T, q);
            double lse_p = sgbv_oracle_softmax(rp, V, T, p);
            R = sgbv_oracle_resmass(q, p, V, 1.0, exp(logb[b] - loga[b]), K, w);
            y = sgbv_oracle_sample(w, V, (double)u[b], &margin);
            if (y < 0) {
                status |= ORACLE_STATUS_DEGENERATE_RESIDUAL;
                y = sgbv_oracle_sample(q, V, (double)u[b], &margin);
                if (out_qnew) memcpy(out_qnew + (size_t)b * V, q, (size_t)V * sizeof(double));
            } else if (out_qnew) {
                for (int x = 0; x < V; ++x) out_qnew[(size_t)b * V + x] = w[x] / R;
            }
            la = loga[b] + ((double)rq[y] / T - lse_q);
            lb = logb[b] + ((double)rp[y] / T - lse_p);
            free(q); free(p); free(w);
        } else if (out_qnew) {
            for (int x = 0; x < V; ++x) out_qnew[(size_t)b * V + x] = NAN;
        }
        out_token[b] = y;
        if (out_loga) out_loga[b] = la;
        if (out_logb) out_logb[b] = lb;
        if (out_R) out_R[b] = R;
        if (out_status) out_status[b] = status;
        if (out_margin) out_margin[b] = margin;
    }
    return 1;
}

/* ============================================================================================== */
/* Comparison verifiers of Section 3: token-level speculative sampling (3.1) and SpecTr's K-SEQ   */
/* (3.2), position by position.  K = 1 of K-SEQ is token-level speculative sampling (rho = 1).     */
/*                                                                                                 */
/* Per position i, with the drafts that still match the accepted prefix ("retained", n of them;    */
/* they share the rows of that prefix, the rows of the first retained draft are read):             */
/*   beta(rho) = sum_x min{p(x), q(x)/rho};  rho in [1, n] solves 1 - (1 - beta(rho))^n = rho beta(rho) */
/*   (bisection; the left side minus the right is >= 0 at rho = 1 and <= 0 at rho = n);            */
/*   the retained drafts are tried in order: draft k's token x is accepted if eta_{k,i} <          */
/*   min{1, q(x)/(rho p(x))}; the first accepted token extends the prefix and the drafts with that */
/*   token stay retained; if none is accepted, y is drawn from norm(q - rho min{p, q/rho}) =       */
/*   norm(max{q - rho p, 0}) and the step ends; after L accepted positions y ~ q(.|x^L).           */
/* Reading: n is the number of retained drafts at that position (the candidates that are actually  */
/* i.i.d. draws from p(.|prefix)), n = K at the first position.                                    */
/* Layouts as in sgbv_oracle_verify; uniforms[b, k*gamma + i] is eta of draft k at position i      */
/* (0-based), the last entry draws y.  out_rho [B,gamma] (NaN where not reached); out_acc          */
/* [B,K,gamma] acceptance probabilities of the tokens that were tried (NaN elsewhere).             */
static double kseq_beta(const double *q, const double *p, int V, double rho) {
    double s = 0.0;
    for (int x = 0; x < V; ++x) {
        double t = q[x] / rho;
        s += p[x] < t ? p[x] : t;
    }
    return s;
}

double sgbv_oracle_kseq_rho(const double *q, const double *p, int V, int n) {
    if (n <= 1) return 1.0;
    double lo = 1.0, hi = (double)n;
    for (int it = 0; it < 200 && hi - lo > 1e-15 * hi; ++it) {
        double mid = 0.5 * (lo + hi);
        double beta = kseq_beta(q, p, V, mid);
        double f = sgbv_oracle_g(beta, n) - mid * beta;
        if (f > 0.0) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

int sgbv_oracle_kseq_verify(const float *zq, const float *zp, const int32_t *tok, const float *uniforms,
                            int B, int K, int gamma, int V, double T, int32_t *out_tau,
                            int32_t *out_tokens, double *out_rho, double *out_acc, int32_t *out_status,
                            double *out_margin_accept, double *out_margin_sample) {
    if (B < 0 || K < 1 || gamma < 1 || V < 1 || !(T > 0.0) || !isfinite(T)) return -1;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int b = 0; b < B; ++b) {
        const float *zq_b = zq + (size_t)b * K * (gamma + 1) * V, *zp_b = zp + (size_t)b * K * gamma * V;
        const int32_t *tok_b = tok + (size_t)b * K * gamma;
        const float *u = uniforms + (size_t)b * (K * gamma + 1);
        double *q = (double *)malloc((size_t)V * sizeof(double));
        double *p = (double *)malloc((size_t)V * sizeof(double));
        double *w = (double *)malloc((size_t)V * sizeof(double));
        int *kept = (int *)malloc((size_t)K * sizeof(int));
        int status = 0;
        for (int n = 0; n < K * gamma; ++n)
            if (tok_b[n] < 0 || tok_b[n] >= V) status |= ORACLE_STATUS_TOKEN_RANGE;
        for (int i = 0; i <= gamma; ++i) out_tokens[(size_t)b * (gamma + 1) + i] = -1;
        for (int i = 0; i < gamma; ++i) out_rho[(size_t)b * gamma + i] = NAN;
        for (int n = 0; n < K * gamma; ++n) out_acc[(size_t)b * K * gamma + n] = NAN;
        int tau = 0;
        int32_t y = -1;
        double margin_a = INFINITY, margin_s = 0.0;
        int nk = K;
        for (int k = 0; k < K; ++k) kept[k] = k;
        int stopped = 0;
        for (int i = 0; i < gamma && status == 0 && !stopped; ++i) {
            const float *rq = zq_b + ((size_t)kept[0] * (gamma + 1) + i) * V;
            const float *rp = zp_b + ((size_t)kept[0] * gamma + i) * V;
            int anyq = 0, anyp = 0;
            for (int x = 0; x < V; ++x) {
                if (isnan(rq[x]) || rq[x] == INFINITY || isnan(rp[x]) || rp[x] == INFINITY)
                    status |= ORACLE_STATUS_NONFINITE;
                anyq |= isfinite(rq[x]);
                anyp |= isfinite(rp[x]);
            }
            if (!anyq || !anyp) status |= ORACLE_STATUS_NONFINITE;
            if (status) break;
            sgbv_oracle_softmax(rq, V, T, q);
            sgbv_oracle_softmax(rp, V, T, p);
            double rho = sgbv_oracle_kseq_rho(q, p, V, nk);
            out_rho[(size_t)b * gamma + i] = rho;
            int accepted = -1;
            for (int j = 0; j < nk && accepted < 0; ++j) {
                int k = kept[j];
                int32_t x = tok_b[k * gamma + i];
                double acc = (p[x] > 0.0) ? q[x] / (rho * p[x]) : 1.0;
                if (acc > 1.0) acc = 1.0;
                out_acc[((size_t)b * K + k) * gamma + i] = acc;
                double eta = (double)u[k * gamma + i];
                double d = fabs(eta - acc);
                if (d < margin_a) margin_a = d;
                if (eta < acc) accepted = k;
            }
            if (accepted >= 0) {
                int32_t x = tok_b[accepted * gamma + i];
                out_tokens[(size_t)b * (gamma + 1) + i] = x;
                tau = i + 1;
                int m = 0;
                for (int j = 0; j < nk; ++j)
                    if (tok_b[kept[j] * gamma + i] == x) kept[m++] = kept[j];
                nk = m;
            } else {
                for (int x = 0; x < V; ++x) {
                    double d = q[x] - rho * p[x];
                    w[x] = d > 0.0 ? d : 0.0;
                }
                y = sgbv_oracle_sample(w, V, (double)u[K * gamma], &margin_s);
                if (y < 0) {
                    status |= ORACLE_STATUS_DEGENERATE_RESIDUAL;
                    y = sgbv_oracle_sample(q, V, (double)u[K * gamma], &margin_s);
                }
                stopped = 1;
            }
        }
        if (status == 0 || status == ORACLE_STATUS_DEGENERATE_RESIDUAL) {
            if (!stopped) { /* every position accepted: bonus token from the target row after the block */
                const float *rq = zq_b + ((size_t)kept[0] * (gamma + 1) + gamma) * V;
                int any = 0, badrow = 0;
                for (int x = 0; x < V; ++x) {
                    badrow |= isnan(rq[x]) || rq[x] == INFINITY;
                    any |= isfinite(rq[x]);
                }
                if (badrow || !any) {
                    status |= ORACLE_STATUS_NONFINITE;
                } else {
                    sgbv_oracle_softmax(rq, V, T, q);
                    y = sgbv_oracle_sample(q, V, (double)u[K * gamma], &margin_s);
                }
            }
        }
        if (status & (ORACLE_STATUS_NONFINITE | ORACLE_STATUS_TOKEN_RANGE)) {
            tau = -1;
            for (int i = 0; i <= gamma; ++i) out_tokens[(size_t)b * (gamma + 1) + i] = -1;
        } else {
            out_tokens[(size_t)b * (gamma + 1) + tau] = y;
        }
        out_tau[b] = tau;
        if (out_status) out_status[b] = status;
        if (out_margin_accept) out_margin_accept[b] = margin_a;
        if (out_margin_sample) out_margin_sample[b] = margin_s;
        free(q); free(p); free(w); free(kept);
    }
    return 1;
}

/* ============================================================================================== */
/* Algorithm 3's draft draw, one position: token r ~ softmax(z[r]/T) by the inverse CDF of step 6.  */
/*   z [N,V]; u [N]; out_token [N] (-1 for a row with NaN/+inf or no finite logit); out_logp [N]    */
/*   (log softmax of the drawn token) and out_margin [N] may be NULL.                               */
int sgbv_oracle_draw_tokens(const float *z, const float *u, int N, int V, double T, int32_t *out_token,
                            double *out_logp, double *out_margin) {
    if (N < 0 || V < 1 || !(T > 0.0) || !isfinite(T)) return -1;
    double *prob = (double *)malloc((size_t)V * sizeof(double));
    for (int r = 0; r < N; ++r) {
        const float *row = z + (size_t)r * V;
        int any = 0, bad = 0;
        for (int x = 0; x < V; ++x) {
            bad |= isnan(row[x]) || row[x] == INFINITY;
            any |= isfinite(row[x]);
        }
        double margin = 0.0, lp = NAN;
        int32_t y = -1;
        if (!bad && any) {
            double lse = sgbv_oracle_softmax(row, V, T, prob);
            y = sgbv_oracle_sample(prob, V, (double)u[r], &margin);
            lp = (double)row[y] / T - lse;
        }
        out_token[r] = y;
        if (out_logp) out_logp[r] = lp;
        if (out_margin) out_margin[r] = margin;
    }
    free(prob);
    return 1;
}
