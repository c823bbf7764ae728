/*
 * CPU oracle for the MeteoRA linear forward.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the plain definition of what the GPU library must compute,
 * written token by token with fp64 accumulation.  It is slow on purpose and
 * shares no code, header, table or helper with the CUDA path.  Only the test
 * suite, the smoke check and the benchmark's cpu_baseline / reference legs may
 * load it; no product code path may call into it.
 *
 * What it follows (paper: "MeteoRA: Multiple-tasks Embedded LoRA for Large
 * Language Models"):
 *   - Sec. 3.1: the gating network G maps a token x in R^d to n logits; the k
 *     adapters with the highest logits form I(x).
 *   - Eq. 3: the weight of a selected adapter is the softmax of its logit over
 *     the selected k logits only.
 *   - Eq. 2: o = x W_base + sum_{i in I(x)} w_i ((x A_i) B_i).
 *   - Eq. 1 / App. A.1 (top-1): k = 1 gives the classical LoRA forward
 *     W_base x + B_i A_i x with weight exactly 1.
 *   - Sec. 3.3 (loop-original): tokens that picked adapter i are gathered into
 *     one group per adapter; the routing function below produces that grouping
 *     as a stable counting sort.
 *   - App. A.5: a temperature divides the selected logits before the softmax.
 *   - Sec. 3.2: only the gating networks are trained; meteora_oracle_gate_backward is the chain rule of Eq. 2
 *     and Eq. 3 with respect to the gate weights.
 *
 * Storage convention (row-major, contiguous; transposes of the paper's
 * (n,d,r) / (n,r,h) tensors so that every contraction runs along the
 * contiguous axis):
 *   x[T,d_in]  W0[d_out,d_in]  A[N,r,d_in]  B[N,d_out,r]  Wg[N,d_in]  y[T,d_out]
 *
 * Precision.  Inputs are float (bf16 workloads are rounded to bf16 by the input
 * generator and arrive here as exactly representable floats).  Every sum is
 * accumulated in double in ascending index order.  The logit is rounded once
 * to float before it is compared, because the selection is an integer decision
 * and the library takes it on fp32 logits.  Outputs stay double.
 *
 * Pins (tests marked "not gpu"): zero B gives the plain matrix product; top-1
 * with a forced gate gives single LoRA; weights sum to one and follow the
 * closed-form two-logit softmax; a hand-worked integer example; relabelling the
 * adapters leaves the output unchanged; evaluating all N adapters under a 0/w
 * gate mask (the batched view of Eq. 5) gives the same result; k = N gives the
 * full softmax mixture; the routing equals a stable argsort.  No function in
 * this file is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_BAD_ARG (-1)
#define ORACLE_MAX_N 4096

int meteora_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void meteora_oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Sec. 3.1: logits of one token, G(x)_n = sum_d Wg[n,d] x[d]; rounded to float once. */
static void token_logits(const float *xt, const float *Wg, int d_in, int N, float *logit) {
    for (int n = 0; n < N; ++n) {
        double acc = 0.0;
        const float *g = Wg + (size_t)n * d_in;
        for (int d = 0; d < d_in; ++d) acc += (double)g[d] * (double)xt[d];
        logit[n] = (float)acc;
    }
}

/* Sec. 3.1: I(x) = the k highest logits, listed by descending logit; equal logits
 * keep the lower adapter index first. */
static void token_topk(const float *logit, int N, int k, int32_t *sel) {
    unsigned char *taken = (unsigned char *)calloc((size_t)N, 1);
    for (int j = 0; j < k; ++j) {
        int best = -1;
        for (int n = 0; n < N; ++n) {
            if (taken[n]) continue;
            if (best < 0 || logit[n] > logit[best]) best = n; /* strict: ties stay at lower n */
        }
        taken[best] = 1;
        sel[j] = best;
    }
    free(taken);
}

/* Eq. 3 with the temperature of App. A.5: w_j = exp(l_j/tau) / sum_{j' in I(x)} exp(l_j'/tau). */
static void token_weights(const float *logit, const int32_t *sel, int k, double tau, double *w) {
    double m = (double)logit[sel[0]];
    for (int j = 1; j < k; ++j)
        if ((double)logit[sel[j]] > m) m = (double)logit[sel[j]];
    double s = 0.0;
    for (int j = 0; j < k; ++j) {
        w[j] = exp(((double)logit[sel[j]] - m) / tau);
        s += w[j];
    }
    for (int j = 0; j < k; ++j) w[j] /= s;
}

/* x W_base of Eq. 2 for one token. */
static void token_base(const float *xt, const float *W0, int d_in, int d_out, double *out) {
    for (int o = 0; o < d_out; ++o) {
        double acc = 0.0;
        const float *wrow = W0 + (size_t)o * d_in;
        for (int d = 0; d < d_in; ++d) acc += (double)wrow[d] * (double)xt[d];
        out[o] = acc;
    }
}

/* sum_{i in I(x)} w_i ((x A_i) B_i) of Eq. 2 for one token, added into out. */
static void token_delta(const float *xt, const float *A, const float *B, const int32_t *sel, const double *w,
                        int d_in, int d_out, int r, int k, double *out) {
    double *u = (double *)malloc(sizeof(double) * (size_t)r);
    for (int j = 0; j < k; ++j) {
        const int i = sel[j];
        const float *Ai = A + (size_t)i * r * d_in;
        const float *Bi = B + (size_t)i * d_out * r;
        for (int p = 0; p < r; ++p) {
            double acc = 0.0;
            for (int d = 0; d < d_in; ++d) acc += (double)Ai[(size_t)p * d_in + d] * (double)xt[d];
            u[p] = acc;
        }
        for (int o = 0; o < d_out; ++o) {
            double acc = 0.0;
            for (int p = 0; p < r; ++p) acc += (double)Bi[(size_t)o * r + p] * u[p];
            out[o] += w[j] * acc;
        }
    }
    free(u);
}

static int bad_dims(int T, int d_in, int N, int k) {
    return T < 0 || d_in <= 0 || N <= 0 || N > ORACLE_MAX_N || k <= 0 || k > N;
}

/* Gate, selection and weights for every token (Sec. 3.1, Eq. 3).
 * topk_idx[T,k] int32, topk_w[T,k] double, logits[T,N] float (may be NULL). */
int meteora_oracle_gate_topk(const float *x, const float *Wg, int T, int d_in, int N, int k, double tau,
                             int32_t *topk_idx, double *topk_w, float *logits) {
    if (bad_dims(T, d_in, N, k) || !(tau > 0.0)) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        float *logit = (float *)malloc(sizeof(float) * (size_t)N);
        token_logits(x + (size_t)t * d_in, Wg, d_in, N, logit);
        token_topk(logit, N, k, topk_idx + (size_t)t * k);
        token_weights(logit, topk_idx + (size_t)t * k, k, tau, topk_w + (size_t)t * k);
        if (logits) memcpy(logits + (size_t)t * N, logit, sizeof(float) * (size_t)N);
        free(logit);
    }
    return ORACLE_OK;
}

/* Grouping of the T*k (token, pick) slots by adapter (Sec. 3.3, the gather of
 * loop-original).  Slot s = t*k + j has key topk_idx[s].  counts[N] is the
 * histogram, offsets[N+1] its exclusive prefix sum, perm[T*k] the slots sorted
 * by key with equal keys in ascending slot order. */
int meteora_oracle_route(const int32_t *topk_idx, int T, int k, int N, int32_t *counts, int32_t *offsets,
                         int32_t *perm) {
    if (T < 0 || k <= 0 || N <= 0) return ORACLE_BAD_ARG;
    const int S = T * k;
    for (int e = 0; e < N; ++e) counts[e] = 0;
    for (int s = 0; s < S; ++s) {
        if (topk_idx[s] < 0 || topk_idx[s] >= N) return ORACLE_BAD_ARG;
        counts[topk_idx[s]] += 1;
    }
    offsets[0] = 0;
    for (int e = 0; e < N; ++e) offsets[e + 1] = offsets[e] + counts[e];
    int32_t *cursor = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    for (int e = 0; e < N; ++e) cursor[e] = offsets[e];
    for (int s = 0; s < S; ++s) perm[cursor[topk_idx[s]]++] = s;
    free(cursor);
    return ORACLE_OK;
}

/* The LoRA term of Eq. 2 alone, for given selections and weights.
 * delta[T,d_out] double. */
int meteora_oracle_lora_delta(const float *x, const float *A, const float *B, const int32_t *topk_idx,
                              const float *topk_w, int T, int d_in, int d_out, int N, int r, int k,
                              double *delta) {
    if (bad_dims(T, d_in, N, k) || d_out <= 0 || r <= 0) return ORACLE_BAD_ARG;
    for (size_t s = 0; s < (size_t)T * k; ++s)
        if (topk_idx[s] < 0 || topk_idx[s] >= N) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        double *w = (double *)malloc(sizeof(double) * (size_t)k);
        for (int j = 0; j < k; ++j) w[j] = (double)topk_w[(size_t)t * k + j];
        double *out = delta + (size_t)t * d_out;
        for (int o = 0; o < d_out; ++o) out[o] = 0.0;
        token_delta(x + (size_t)t * d_in, A, B, topk_idx + (size_t)t * k, w, d_in, d_out, r, k, out);
        free(w);
    }
    return ORACLE_OK;
}

/* The whole layer, Eq. 2 with Eq. 3: gate, select, weigh, base product, LoRA sum.
 * y[T,d_out] double; topk_idx / topk_w receive the routing that was used (may be NULL). */
int meteora_oracle_linear_forward(const float *x, const float *W0, const float *A, const float *B,
                                  const float *Wg, int T, int d_in, int d_out, int N, int r, int k, double tau,
                                  double *y, int32_t *topk_idx, double *topk_w) {
    if (bad_dims(T, d_in, N, k) || d_out <= 0 || r <= 0 || !(tau > 0.0)) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        const float *xt = x + (size_t)t * d_in;
        float *logit = (float *)malloc(sizeof(float) * (size_t)N);
        int32_t *sel = (int32_t *)malloc(sizeof(int32_t) * (size_t)k);
        double *w = (double *)malloc(sizeof(double) * (size_t)k);
        token_logits(xt, Wg, d_in, N, logit);
        token_topk(logit, N, k, sel);
        token_weights(logit, sel, k, tau, w);
        token_base(xt, W0, d_in, d_out, y + (size_t)t * d_out);
        token_delta(xt, A, B, sel, w, d_in, d_out, r, k, y + (size_t)t * d_out);
        if (topk_idx) memcpy(topk_idx + (size_t)t * k, sel, sizeof(int32_t) * (size_t)k);
        if (topk_w) memcpy(topk_w + (size_t)t * k, w, sizeof(double) * (size_t)k);
        free(logit);
        free(sel);
        free(w);
    }
    return ORACLE_OK;
}

/* Eq. 2 with the selection given from outside: the weights are still Eq. 3 on
 * this side's logits of the given adapters.  Used where two selections are both
 * valid (logits closer than the comparison band) to check the output that
 * belongs to the other side's selection. */
int meteora_oracle_linear_forward_routed(const float *x, const float *W0, const float *A, const float *B,
                                         const float *Wg, const int32_t *topk_idx, int T, int d_in, int d_out,
                                         int N, int r, int k, double tau, double *y) {
    if (bad_dims(T, d_in, N, k) || d_out <= 0 || r <= 0 || !(tau > 0.0)) return ORACLE_BAD_ARG;
    for (size_t s = 0; s < (size_t)T * k; ++s)
        if (topk_idx[s] < 0 || topk_idx[s] >= N) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        const float *xt = x + (size_t)t * d_in;
        float *logit = (float *)malloc(sizeof(float) * (size_t)N);
        double *w = (double *)malloc(sizeof(double) * (size_t)k);
        token_logits(xt, Wg, d_in, N, logit);
        token_weights(logit, topk_idx + (size_t)t * k, k, tau, w);
        token_base(xt, W0, d_in, d_out, y + (size_t)t * d_out);
        token_delta(xt, A, B, topk_idx + (size_t)t * k, w, d_in, d_out, r, k, y + (size_t)t * d_out);
        free(logit);
        free(w);
    }
    return ORACLE_OK;
}

/*
 * Gradient of the gating network's weights (Sec. 3.2: the base model and the adapters stay fixed, only the
 * gating networks are trained; with top-k > 1 the token loss reaches them through the weights of Eq. 3).
 * Given dy = dL/dy and a selection, by the chain rule on Eq. 2 and Eq. 3 (temperature of App. A.5):
 *     v_j        = (x A_{i_j}) B_{i_j}                      the adapter's own output, in R^{d_out}
 *     g_j        = < dy, v_j >                             = dL/dw_j
 *     dlogit_j   = w_j (g_j - sum_m w_m g_m) / tau         softmax over the selected logits
 *     dWg[i_j,:] += dlogit_j * x                           G(x) = Wg x
 * summed over the tokens.  Unselected adapters get no gradient from this path.  fp64 throughout; the weights
 * are recomputed from this side's logits for the given selection, as in the routed forward.
 */
int meteora_oracle_gate_backward(const float *x, const float *A, const float *B, const float *Wg, const float *dy,
                                 const int32_t *topk_idx, int T, int d_in, int d_out, int N, int r, int k,
                                 double tau, double *dlogit, double *dWg) {
    if (bad_dims(T, d_in, N, k) || d_out <= 0 || r <= 0 || !(tau > 0.0)) return ORACLE_BAD_ARG;
    for (size_t s = 0; s < (size_t)T * k; ++s)
        if (topk_idx[s] < 0 || topk_idx[s] >= N) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        const float *xt = x + (size_t)t * d_in;
        const float *dyt = dy + (size_t)t * d_out;
        const int32_t *sel = topk_idx + (size_t)t * k;
        float *logit = (float *)malloc(sizeof(float) * (size_t)N);
        double *w = (double *)malloc(sizeof(double) * (size_t)k);
        double *g = (double *)malloc(sizeof(double) * (size_t)k);
        double *u = (double *)malloc(sizeof(double) * (size_t)r);
        token_logits(xt, Wg, d_in, N, logit);
        token_weights(logit, sel, k, tau, w);
        for (int j = 0; j < k; ++j) {
            const float *Ai = A + (size_t)sel[j] * r * d_in;
            const float *Bi = B + (size_t)sel[j] * d_out * r;
            for (int p = 0; p < r; ++p) {
                double acc = 0.0;
                for (int d = 0; d < d_in; ++d) acc += (double)Ai[(size_t)p * d_in + d] * (double)xt[d];
                u[p] = acc;
            }
            double gj = 0.0;
            for (int o = 0; o < d_out; ++o) {
                double v = 0.0;
                for (int p = 0; p < r; ++p) v += (double)Bi[(size_t)o * r + p] * u[p];
                gj += (double)dyt[o] * v;
            }
            g[j] = gj;
        }
        double mean = 0.0;
        for (int j = 0; j < k; ++j) mean += w[j] * g[j];
        for (int j = 0; j < k; ++j) dlogit[(size_t)t * k + j] = w[j] * (g[j] - mean) / tau;
        free(logit);
        free(w);
        free(g);
        free(u);
    }
    for (size_t i = 0; i < (size_t)N * d_in; ++i) dWg[i] = 0.0;
    for (int t = 0; t < T; ++t)                                  /* in token order: one writer per row at a time */
        for (int j = 0; j < k; ++j) {
            double *row = dWg + (size_t)topk_idx[(size_t)t * k + j] * d_in;
            const double dl = dlogit[(size_t)t * k + j];
            for (int d = 0; d < d_in; ++d) row[d] += dl * (double)x[(size_t)t * d_in + d];
        }
    return ORACLE_OK;
}
