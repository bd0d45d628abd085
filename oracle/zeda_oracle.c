/*
 * CPU oracle for the zero-expert MoE layer forward (ZEDA).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what
 * the layer computes, written from the paper's definitions.  It shares no code
 * with the CUDA library and must never be reached from the product path; only
 * the tests, the smoke check and the benchmark's CPU-baseline leg call it.
 *
 * What it follows:
 *   - Section 2.1 "Zero-Expert Injection": N normal experts, N_Z zero experts
 *     with Z_j(h) = 0, top-K chosen from the union, K unchanged.
 *   - Eq. 1: y~(h) = sum over selected slots that are normal experts of
 *     g~_i(h) E_i(h); the weights of the surviving slots are NOT rescaled
 *     (Section 4.3.4, text before Eq. 7).
 *   - Eq. 7: the renormalised variant divides by the sum of the weights of
 *     the selected normal experts.
 *   - Appendix B: the copy-expert variant adds (sum of zero-slot weights) * h.
 *   - Appendix D: each expert has up, gate and down projections.
 *   - Eq. 4-6: f_i, P_i, L_A, L_GA forward values.
 *
 * Readings taken where the paper is silent:
 *   score function softmax; "normalised routing weight" = softmax restricted to
 *   the K selected logits (mode 0) or the raw softmax entry (mode 1); top-K ties
 *   go to the lower index; expert = down(silu(gate x) * up x) without biases;
 *   optional additive router bias; logits are rounded once to fp32 and every
 *   later decision uses those fp32 values.
 *
 * Arithmetic: fp64 accumulation everywhere, no blocking or reordering: every
 * sum runs over its index in increasing order.  bf16 inputs arrive as raw
 * 16-bit patterns.
 *
 * Pins (tests/test_oracle_*.py): brute-force top-K on tiny cases, gate-weight
 * invariants, Z=0 against an independent static MoE, all-zero token -> exact 0,
 * Eq. 7 and Appendix-B identities, dense-mask second formulation, plain SwiGLU
 * MLP special case, stable sort against a library stable argsort.  The choice
 * between gate modes 0 and 1 has no numeric example in the paper: for that
 * choice, parity unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { GATE_TOPK_NORM = 0, GATE_SOFTMAX_RAW = 1, GATE_RENORM_REAL = 2 };
enum { EXPERT_ZERO = 0, EXPERT_COPY = 1 };

static double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int zeda_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Router logits over the N + N_Z candidates (Section 2.1): l[t,j] = <x_t, W_r[j]> + b[j],
 * summed in fp64 in increasing feature order, rounded once to fp32. */
void zeda_oracle_logits(const uint16_t *x, const float *router_w, const float *router_bias,
                        int T, int d, int n_cand, float *logits) {
    for (int t = 0; t < T; ++t) {
        for (int j = 0; j < n_cand; ++j) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c)
                acc += bf16_to_double(x[(size_t)t * d + c]) * (double)router_w[(size_t)j * d + c];
            if (router_bias) acc += (double)router_bias[j];
            logits[(size_t)t * n_cand + j] = (float)acc;
        }
    }
}

/* Top-K set "selected from E'" (Section 2.1) for one token, as K rounds of
 * argmax over the not-yet-chosen candidates; equal logits go to the lower
 * index.  Then the routing weights g~ for the K slots. */
static void route_one(const float *l, int n_real, int n_zero, int K, int gate_mode,
                      int32_t *idx, double *w) {
    const int n = n_real + n_zero;
    for (int k = 0; k < K; ++k) {
        int best = -1;
        for (int j = 0; j < n; ++j) {
            int taken = 0;
            for (int q = 0; q < k; ++q) taken |= (idx[q] == j);
            if (taken) continue;
            if (best < 0 || l[j] > l[best]) best = j; /* strict >: lower index wins ties */
        }
        idx[k] = best;
    }
    /* softmax over all candidates, max-subtracted, fp64 */
    double m = (double)l[0];
    for (int j = 1; j < n; ++j) if ((double)l[j] > m) m = (double)l[j];
    double denom_all = 0.0;
    for (int j = 0; j < n; ++j) denom_all += exp((double)l[j] - m);
    double sum_sel = 0.0, sum_real = 0.0;
    for (int k = 0; k < K; ++k) {
        double p = exp((double)l[idx[k]] - m) / denom_all;
        w[k] = p;
        sum_sel += p;
        if (idx[k] < n_real) sum_real += p;
    }
    if (gate_mode == GATE_TOPK_NORM) {
        /* normalised over the K selected slots, zero-expert slots included */
        for (int k = 0; k < K; ++k) w[k] /= sum_sel;
    } else if (gate_mode == GATE_RENORM_REAL) {
        /* Eq. 7: rescaled to sum to one over the selected normal experts */
        for (int k = 0; k < K; ++k)
            w[k] = (idx[k] < n_real && sum_real > 0.0) ? w[k] / sum_real : 0.0;
    } /* GATE_SOFTMAX_RAW: keep p */
}

void zeda_oracle_route(const float *logits, int T, int n_real, int n_zero, int K, int gate_mode,
                       int32_t *topk_idx, double *topk_w) {
    const int n = n_real + n_zero;
    for (int t = 0; t < T; ++t)
        route_one(logits + (size_t)t * n, n_real, n_zero, K, gate_mode,
                  topk_idx + (size_t)t * K, topk_w + (size_t)t * K);
}

/* Dropping the zero-expert slots and grouping the surviving (token, expert)
 * pairs by expert: counts, exclusive offsets and the order (expert ascending,
 * then token ascending), each pair named by its source slot t*K+k.
 * Returns P, the number of surviving pairs. */
int zeda_oracle_compact(const int32_t *topk_idx, int T, int n_real, int K,
                        int32_t *counts, int32_t *offsets, int32_t *perm) {
    for (int e = 0; e < n_real; ++e) counts[e] = 0;
    for (int s = 0; s < T * K; ++s)
        if (topk_idx[s] < n_real) counts[topk_idx[s]]++;
    offsets[0] = 0;
    for (int e = 0; e < n_real; ++e) offsets[e + 1] = offsets[e] + counts[e];
    int p = 0;
    for (int e = 0; e < n_real; ++e)
        for (int t = 0; t < T; ++t)
            for (int k = 0; k < K; ++k)
                if (topk_idx[t * K + k] == e) perm[p++] = t * K + k;
    return p;
}

/* One normal expert applied to one token (Appendix D: up, gate and down
 * projections; SwiGLU reading): o = W_down (silu(W_gate x) * (W_up x)).
 * w_gate_up is [2*He, d] (gate rows first), w_down is [d, He]. */
static void expert_one(const double *xd, const uint16_t *w_gate_up, const uint16_t *w_down,
                       int d, int He, double *hmid, double *o) {
    for (int j = 0; j < He; ++j) {
        double a = 0.0, u = 0.0;
        const uint16_t *wg = w_gate_up + (size_t)j * d;
        const uint16_t *wu = w_gate_up + (size_t)(He + j) * d;
        for (int c = 0; c < d; ++c) {
            a += bf16_to_double(wg[c]) * xd[c];
            u += bf16_to_double(wu[c]) * xd[c];
        }
        hmid[j] = a / (1.0 + exp(-a)) * u;
    }
    for (int c = 0; c < d; ++c) {
        double acc = 0.0;
        const uint16_t *wd = w_down + (size_t)c * He;
        for (int j = 0; j < He; ++j) acc += bf16_to_double(wd[j]) * hmid[j];
        o[c] = acc;
    }
}

void zeda_oracle_expert(const uint16_t *x_row, const uint16_t *w_gate_up_e, const uint16_t *w_down_e,
                        int d, int He, double *o) {
    double *xd = (double *)malloc(sizeof(double) * d);
    double *hm = (double *)malloc(sizeof(double) * He);
    for (int c = 0; c < d; ++c) xd[c] = bf16_to_double(x_row[c]);
    expert_one(xd, w_gate_up_e, w_down_e, d, He, hm, o);
    free(xd);
    free(hm);
}

/* Full layer forward for the listed tokens (Eq. 1; Eq. 7 through gate_mode;
 * Appendix B through expert_kind).  token_ids == NULL means tokens 0..n_tok-1.
 * Every token is independent of the others, so a subset is exact.
 * Outputs (any may be NULL): y [n_tok, d] fp64, idx [n_tok, K], w [n_tok, K]. */
void zeda_oracle_forward(const uint16_t *x, int d, int He, int n_real, int n_zero, int K,
                         int gate_mode, int expert_kind,
                         const float *router_w, const float *router_bias,
                         const uint16_t *w_gate_up, const uint16_t *w_down,
                         const int32_t *token_ids, int n_tok,
                         double *y, int32_t *topk_idx, double *topk_w) {
    const int n = n_real + n_zero;
#pragma omp parallel
    {
        float *l = (float *)malloc(sizeof(float) * n);
        int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * K);
        double *w = (double *)malloc(sizeof(double) * K);
        double *xd = (double *)malloc(sizeof(double) * d);
        double *hm = (double *)malloc(sizeof(double) * He);
        double *o = (double *)malloc(sizeof(double) * d);
#pragma omp for schedule(dynamic, 1)
        for (int i = 0; i < n_tok; ++i) {
            const int t = token_ids ? token_ids[i] : i;
            const uint16_t *xt = x + (size_t)t * d;
            zeda_oracle_logits(xt, router_w, router_bias, 1, d, n, l);
            route_one(l, n_real, n_zero, K, gate_mode, idx, w);
            for (int c = 0; c < d; ++c) xd[c] = bf16_to_double(xt[c]);
            if (y) {
                double *yt = y + (size_t)i * d;
                for (int c = 0; c < d; ++c) yt[c] = 0.0;
                for (int k = 0; k < K; ++k) {
                    if (idx[k] < n_real) {
                        const int e = idx[k];
                        expert_one(xd, w_gate_up + (size_t)e * 2 * He * d,
                                   w_down + (size_t)e * d * He, d, He, hm, o);
                        for (int c = 0; c < d; ++c) yt[c] += w[k] * o[c];
                    } else if (expert_kind == EXPERT_COPY) {
                        for (int c = 0; c < d; ++c) yt[c] += w[k] * xd[c];
                    }
                }
            }
            if (topk_idx) memcpy(topk_idx + (size_t)i * K, idx, sizeof(int32_t) * K);
            if (topk_w) memcpy(topk_w + (size_t)i * K, w, sizeof(double) * K);
        }
        free(l); free(idx); free(w); free(xd); free(hm); free(o);
    }
}

/* Routing statistics and regulariser forward values over a batch (Eq. 4-6).
 * f[i]  = fraction of tokens whose top-K set contains candidate i,
 * pm[i] = mean routing probability of candidate i; the paper calls P_i "the
 *         mean routing probability assigned to expert i", read here as the
 *         softmax probability over all N+N_Z candidates (selected or not), the
 *         form of the load-balancing loss the paper derives L_A from,
 * out[0] = r_ZE (share of the T*K slots that landed on zero experts),
 * out[1] = L_A  = alpha (N+N_Z)/K sum_i f_i P_i,
 * out[2] = L_GA = alpha (N+N_Z w)/K (f_E P_E / N + f_Z P_Z / (N_Z w)). */
void zeda_oracle_stats(const float *logits, const int32_t *topk_idx, int T, int n_real, int n_zero,
                       int K, double alpha, double group_w, double *f, double *pm, double *out) {
    const int n = n_real + n_zero;
    for (int i = 0; i < n; ++i) { f[i] = 0.0; pm[i] = 0.0; }
    long zero_slots = 0;
    for (int t = 0; t < T; ++t) {
        const float *l = logits + (size_t)t * n;
        double m = (double)l[0];
        for (int j = 1; j < n; ++j) if ((double)l[j] > m) m = (double)l[j];
        double denom = 0.0;
        for (int j = 0; j < n; ++j) denom += exp((double)l[j] - m);
        for (int j = 0; j < n; ++j) pm[j] += exp((double)l[j] - m) / denom;
        for (int k = 0; k < K; ++k) {
            int i = topk_idx[(size_t)t * K + k];
            f[i] += 1.0;
            if (i >= n_real) zero_slots++;
        }
    }
    for (int i = 0; i < n; ++i) { f[i] /= T; pm[i] /= T; }
    double la = 0.0, fE = 0.0, pE = 0.0, fZ = 0.0, pZ = 0.0;
    for (int i = 0; i < n; ++i) {
        la += f[i] * pm[i];
        if (i < n_real) { fE += f[i]; pE += pm[i]; } else { fZ += f[i]; pZ += pm[i]; }
    }
    out[0] = (double)zero_slots / ((double)T * K);
    out[1] = alpha * (double)n / K * la;
    double ga = fE * pE / n_real;
    if (n_zero > 0) ga += fZ * pZ / (n_zero * group_w);
    out[2] = alpha * (n_real + n_zero * group_w) / K * ga;
}

/* Per-token zero-expert ratio: the share of token t's K slots that landed on zero experts
 * (Section 2.2 defines r_ZE as the fraction of activated experts that are zero experts; Section 4.1
 * looks at it token by token). */
void zeda_oracle_token_zero_share(const int32_t *topk_idx, int T, int n_real, int K, double *out) {
    for (int t = 0; t < T; ++t) {
        int zero = 0;
        for (int k = 0; k < K; ++k)
            if (topk_idx[(size_t)t * K + k] >= n_real) zero++;
        out[t] = (double)zero / (double)K;
    }
}
