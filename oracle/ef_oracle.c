/*
 * CPU oracle for the five fused tensor programs.  TEST INFRASTRUCTURE ONLY:
 * this file is imported by the tests, by the smoke check and by the benchmark's
 * cpu_baseline leg; the product (the CUDA library) never calls it and shares no
 * code, header, table or helper with it.
 *
 * Every function evaluates the UNFUSED tensor-level definition of its program
 * in fp64: the "M0" form of Figure 4 for attention, and the composite-operator
 * expansions the paper's frontend performs (Section 7.1: RMSNorm and attention
 * are expanded into matmul + reduce + pointwise).  No tiling, no rolling
 * reducer, no factor motion, no reassociation: those are what the CUDA path
 * does and what the tests compare against this.
 *
 * All tensors are row-major, contiguous, last dimension fastest, passed as
 * double (the harness widens bf16 bit patterns exactly).  Outputs are
 * unrounded fp64.  OpenMP parallelises the outermost independent index only.
 *
 * Parity pins (tests/test_oracle_pins.py): every function below is pinned by
 * closed forms, invariants, library special cases and brute force; none is
 * "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int ef_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Inverse root-mean-square of one row of length n: 1/sqrt(mean(x^2) + eps).
 * eps is added to the mean, inside the square root. */
static double inv_rms(const double *x, int n, double eps) {
    double ss = 0.0;
    for (int k = 0; k < n; ++k) ss += x[k] * x[k];
    return 1.0 / sqrt(ss / (double)n + eps);
}

/* out[n] = sum_k a[k] * W[k,n]; loop order k,n so the inner loop streams W rows. */
static void row_times_matrix(const double *a, const double *W, double *out, int K, int N) {
    for (int n = 0; n < N; ++n) out[n] = 0.0;
    for (int k = 0; k < K; ++k) {
        const double ak = a[k];
        const double *w = W + (size_t)k * N;
        for (int n = 0; n < N; ++n) out[n] += ak * w[n];
    }
}

/* Program 1 (Section 7.2, RMSNorm followed by a projection):
 *   r_i = 1/sqrt(mean_k x_ik^2 + eps);  xn_ik = x_ik * r_i * gamma_k;  Y = xn @ W.
 * X [M,K], gamma [K], W [K,N] -> Y [M,N]. */
void ef_oracle_rmsnorm_matmul(const double *X, const double *gamma, const double *W, double *Y,
                              int M, int K, int N, double eps) {
#pragma omp parallel for schedule(static)
    for (int i = 0; i < M; ++i) {
        double *xn = (double *)malloc((size_t)K * sizeof(double));
        const double *x = X + (size_t)i * K;
        const double r = inv_rms(x, K, eps);
        for (int k = 0; k < K; ++k) xn[k] = x[k] * r * gamma[k];
        row_times_matrix(xn, W, Y + (size_t)i * N, K, N);
        free(xn);
    }
}

/* LayerNorm followed by a projection (the LayerNorm+GEMM workload, Sections 7.1 and 7.2; the paper does not
 * define the operator: standard LayerNorm, biased variance, eps inside the square root):
 *   mu_i = mean_k x_ik;  var_i = mean_k (x_ik - mu_i)^2;  xn_ik = (x_ik - mu_i) / sqrt(var_i + eps) * gamma_k + beta_k;
 *   Y = xn @ W.   X [M,K], gamma [K], beta [K], W [K,N] -> Y [M,N]. */
void ef_oracle_layernorm_matmul(const double *X, const double *gamma, const double *beta, const double *W, double *Y,
                                int M, int K, int N, double eps) {
#pragma omp parallel for schedule(static)
    for (int i = 0; i < M; ++i) {
        double *xn = (double *)malloc((size_t)K * sizeof(double));
        const double *x = X + (size_t)i * K;
        double mu = 0.0;
        for (int k = 0; k < K; ++k) mu += x[k];
        mu /= (double)K;
        double var = 0.0;
        for (int k = 0; k < K; ++k) var += (x[k] - mu) * (x[k] - mu);
        var /= (double)K;
        const double r = 1.0 / sqrt(var + eps);
        for (int k = 0; k < K; ++k) xn[k] = (x[k] - mu) * r * gamma[k] + beta[k];
        row_times_matrix(xn, W, Y + (size_t)i * N, K, N);
        free(xn);
    }
}

/* SiLU(z) = z * sigmoid(z), evaluated without overflow for either sign. */
static double silu(double z) {
    if (z >= 0.0) return z / (1.0 + exp(-z));
    const double e = exp(z);
    return z * e / (1.0 + e);
}

/* Program 2 (gated MLP, Section 7.2): G = X@Wgate, U = X@Wup, Y = SiLU(G) * U.
 * X [M,K], Wgate/Wup [K,N] -> Y [M,N]. */
void ef_oracle_gated_mlp(const double *X, const double *Wgate, const double *Wup, double *Y,
                         int M, int K, int N) {
#pragma omp parallel for schedule(static)
    for (int i = 0; i < M; ++i) {
        double *g = (double *)malloc((size_t)N * sizeof(double));
        double *u = (double *)malloc((size_t)N * sizeof(double));
        row_times_matrix(X + (size_t)i * K, Wgate, g, K, N);
        row_times_matrix(X + (size_t)i * K, Wup, u, K, N);
        for (int n = 0; n < N; ++n) Y[(size_t)i * N + n] = silu(g[n]) * u[n];
        free(g);
        free(u);
    }
}

/* Program 2b (RMSNorm-MLP, Section 7.2): the unfused chain RMSNorm -> two projections -> gate:
 *   xn_ik = x_ik * r_i * gamma_k;  G = xn @ Wgate;  U = xn @ Wup;  Y = SiLU(G) * U. */
void ef_oracle_rmsnorm_gated_mlp(const double *X, const double *gamma, const double *Wgate, const double *Wup,
                                 double *Y, int M, int K, int N, double eps) {
#pragma omp parallel for schedule(static)
    for (int i = 0; i < M; ++i) {
        double *xn = (double *)malloc((size_t)K * sizeof(double));
        double *g = (double *)malloc((size_t)N * sizeof(double));
        double *u = (double *)malloc((size_t)N * sizeof(double));
        const double *x = X + (size_t)i * K;
        const double r = inv_rms(x, K, eps);
        for (int k = 0; k < K; ++k) xn[k] = x[k] * r * gamma[k];
        row_times_matrix(xn, Wgate, g, K, N);
        row_times_matrix(xn, Wup, u, K, N);
        for (int n = 0; n < N; ++n) Y[(size_t)i * N + n] = silu(g[n]) * u[n];
        free(xn);
        free(g);
        free(u);
    }
}

/* Vanilla attention of ONE query row against n_keys keys (Figure 4, M0):
 *   score = q.k_j (f32-accumulated matmul in the paper; fp64 here), scaled = score*scale,
 *   maximum = max_j scaled, weights = exp(scaled - maximum), normalizer = sum_j weights,
 *   prob = weights / normalizer, output = prob @ V.
 * keys/values are [n_keys, D] with row stride `stride`. `s` is scratch of n_keys doubles. */
static void attend_row(const double *q, const double *Kmat, const double *Vmat, size_t stride,
                       int n_keys, int D, double scale, double *s, double *out) {
    double mx = -INFINITY;
    for (int j = 0; j < n_keys; ++j) {
        const double *k = Kmat + (size_t)j * stride;
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += q[d] * k[d];
        s[j] = dot * scale;
        if (s[j] > mx) mx = s[j];
    }
    double norm = 0.0;
    for (int j = 0; j < n_keys; ++j) {
        s[j] = exp(s[j] - mx);
        norm += s[j];
    }
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    for (int j = 0; j < n_keys; ++j) {
        const double p = s[j] / norm;
        const double *v = Vmat + (size_t)j * stride;
        for (int d = 0; d < D; ++d) out[d] += p * v[d];
    }
}

/* Program 3 (decode attention, one query token, grouped-query heads):
 * Q [B,Hq,D], K/V [B,Hkv,L,D] -> O [B,Hq,D]; query head h reads kv head h / (Hq/Hkv)
 * (consecutive query heads share a kv head).  The single query is the last position,
 * so all L keys are visible and no mask applies. */
void ef_oracle_gqa_decode(const double *Q, const double *K, const double *V, double *O,
                          int B, int Hq, int Hkv, int L, int D, double scale) {
    const int group = Hq / Hkv;
#pragma omp parallel for schedule(static)
    for (int bh = 0; bh < B * Hq; ++bh) {
        const int b = bh / Hq, h = bh % Hq, g = h / group;
        double *s = (double *)malloc((size_t)L * sizeof(double));
        const size_t kv_off = ((size_t)b * Hkv + g) * (size_t)L * D;
        attend_row(Q + (size_t)bh * D, K + kv_off, V + kv_off, (size_t)D, L, D, scale, s,
                   O + (size_t)bh * D);
        free(s);
    }
}

/* Program 3c (decode attention over a sliding window with attention sinks, Section 7.3): the query is the last
 * position L - 1; key j is visible iff window == 0 or window >= L or j >= L - window or j < sinks.  Softmax and the
 * weighted sum run over the visible keys only (they are gathered first, then Program 3's row routine is applied). */
void ef_oracle_gqa_decode_window(const double *Q, const double *K, const double *V, double *O,
                                 int B, int Hq, int Hkv, int L, int D, double scale, int window, int sinks) {
    const int group = Hq / Hkv;
    const int windowed = window > 0 && window < L;
#pragma omp parallel for schedule(static)
    for (int bh = 0; bh < B * Hq; ++bh) {
        const int b = bh / Hq, h = bh % Hq, g = h / group;
        const size_t kv_off = ((size_t)b * Hkv + g) * (size_t)L * D;
        double *kk = (double *)malloc((size_t)L * D * sizeof(double));
        double *vv = (double *)malloc((size_t)L * D * sizeof(double));
        double *s = (double *)malloc((size_t)L * sizeof(double));
        int n = 0;
        for (int j = 0; j < L; ++j) {
            if (windowed && !(j >= L - window || j < sinks)) continue;
            memcpy(kk + (size_t)n * D, K + kv_off + (size_t)j * D, (size_t)D * sizeof(double));
            memcpy(vv + (size_t)n * D, V + kv_off + (size_t)j * D, (size_t)D * sizeof(double));
            ++n;
        }
        attend_row(Q + (size_t)bh * D, kk, vv, (size_t)D, n, D, scale, s, O + (size_t)bh * D);
        free(kk); free(vv); free(s);
    }
}

/* Program 3b (decode attention, per-sequence key lengths): batch entry b attends keys [0, len_b) of its
 * K/V rows (len_b clamped to [0, L]); rows at and beyond len_b are padding and are never read.  An entry
 * with no keys has no softmax; its output is defined as zero.  Otherwise exactly Program 3 per entry. */
void ef_oracle_gqa_decode_varlen(const double *Q, const double *K, const double *V, const int *lens, double *O,
                                 int B, int Hq, int Hkv, int L, int D, double scale) {
    const int group = Hq / Hkv;
#pragma omp parallel for schedule(static)
    for (int bh = 0; bh < B * Hq; ++bh) {
        const int b = bh / Hq, h = bh % Hq, g = h / group;
        int len = lens[b];
        if (len < 0) len = 0;
        if (len > L) len = L;
        double *out = O + (size_t)bh * D;
        if (len == 0) {
            for (int d = 0; d < D; ++d) out[d] = 0.0;
            continue;
        }
        double *s = (double *)malloc((size_t)len * sizeof(double));
        const size_t kv_off = ((size_t)b * Hkv + g) * (size_t)L * D;
        attend_row(Q + (size_t)bh * D, K + kv_off, V + kv_off, (size_t)D, len, D, scale, s, out);
        free(s);
    }
}

/* Program 4 (prefill attention with RMS-normalised queries and keys):
 *   qh_i = q_i * inv_rms(q_i) * gamma_q;  kh_j = k_j * inv_rms(k_j) * gamma_k  (over head_dim),
 *   then vanilla attention (M0) per (b,h), row i attending keys j <= i when causal.
 * Q,K,V [B,H,S,D], gamma_q/gamma_k [D] (shared by all heads) -> O [B,H,S,D]. */
void ef_oracle_qknorm_attn(const double *Q, const double *K, const double *V,
                           const double *gamma_q, const double *gamma_k, double *O,
                           int B, int H, int S, int D, double eps, double scale, int causal) {
    for (int bh = 0; bh < B * H; ++bh) {
        const size_t off = (size_t)bh * S * D;
        double *kh = (double *)malloc((size_t)S * D * sizeof(double));
#pragma omp parallel for schedule(static)
        for (int j = 0; j < S; ++j) {
            const double *k = K + off + (size_t)j * D;
            const double r = inv_rms(k, D, eps);
            for (int d = 0; d < D; ++d) kh[(size_t)j * D + d] = k[d] * r * gamma_k[d];
        }
#pragma omp parallel for schedule(dynamic, 16)
        for (int i = 0; i < S; ++i) {
            double *s = (double *)malloc((size_t)S * sizeof(double));
            double *qh = (double *)malloc((size_t)D * sizeof(double));
            const double *q = Q + off + (size_t)i * D;
            const double r = inv_rms(q, D, eps);
            for (int d = 0; d < D; ++d) qh[d] = q[d] * r * gamma_q[d];
            const int n_keys = causal ? i + 1 : S;
            attend_row(qh, kh, V + off, (size_t)D, n_keys, D, scale, s, O + off + (size_t)i * D);
            free(s);
            free(qh);
        }
        free(kh);
    }
}

/* Program 4b (Program 4 with grouped KV heads, a sliding window and attention sinks; the mask variants of
 * Section 7.3).  Query head h of batch b reads kv head h / (Hq/Hkv).  With causal != 0 key j is visible to query i
 * iff j <= i and (window == 0 or j > i - window or j < sinks); with causal == 0 every key is visible (window and
 * sinks are then ignored).  Softmax runs over the visible keys only.  Q,O [B,Hq,S,D], K,V [B,Hkv,S,D]. */
void ef_oracle_qknorm_attn_ex(const double *Q, const double *K, const double *V,
                              const double *gamma_q, const double *gamma_k, double *O,
                              int B, int Hq, int Hkv, int S, int D, double eps, double scale, int causal,
                              int window, int sinks) {
    const int group = Hq / Hkv;
    for (int bh = 0; bh < B * Hq; ++bh) {
        const int b = bh / Hq, h = bh % Hq, g = h / group;
        const size_t qoff = (size_t)bh * S * D, koff = ((size_t)b * Hkv + g) * (size_t)S * D;
        double *kh = (double *)malloc((size_t)S * D * sizeof(double));
#pragma omp parallel for schedule(static)
        for (int j = 0; j < S; ++j) {
            const double *k = K + koff + (size_t)j * D;
            const double r = inv_rms(k, D, eps);
            for (int d = 0; d < D; ++d) kh[(size_t)j * D + d] = k[d] * r * gamma_k[d];
        }
#pragma omp parallel for schedule(dynamic, 16)
        for (int i = 0; i < S; ++i) {
            double *s = (double *)malloc((size_t)S * sizeof(double));
            double *qh = (double *)malloc((size_t)D * sizeof(double));
            const double *q = Q + qoff + (size_t)i * D;
            const double r = inv_rms(q, D, eps);
            for (int d = 0; d < D; ++d) qh[d] = q[d] * r * gamma_q[d];
            double mx = -INFINITY;
            for (int j = 0; j < S; ++j) {
                const int vis = !causal || (j <= i && (window == 0 || j > i - window || j < sinks));
                if (!vis) { s[j] = -INFINITY; continue; }
                double dot = 0.0;
                for (int d = 0; d < D; ++d) dot += qh[d] * kh[(size_t)j * D + d];
                s[j] = dot * scale;
                if (s[j] > mx) mx = s[j];
            }
            double norm = 0.0;
            for (int j = 0; j < S; ++j) {
                s[j] = (s[j] == -INFINITY) ? 0.0 : exp(s[j] - mx);
                norm += s[j];
            }
            double *out = O + qoff + (size_t)i * D;
            for (int d = 0; d < D; ++d) out[d] = 0.0;
            for (int j = 0; j < S; ++j) {
                if (s[j] == 0.0) continue;
                const double pj = s[j] / norm;
                const double *v = V + koff + (size_t)j * D;
                for (int d = 0; d < D; ++d) out[d] += pj * v[d];
            }
            free(s);
            free(qh);
        }
        free(kh);
    }
}

/* Program 5 (LoRA-fused linear, Section 7.2): T = X@A;  Y = X@W + alpha * (T@B).
 * X [M,K], W [K,N], A [K,R], Bm [R,N] -> Y [M,N]; alpha multiplies directly. */
void ef_oracle_lora_linear(const double *X, const double *W, const double *A, const double *Bm,
                           double *Y, int M, int K, int N, int R, double alpha) {
#pragma omp parallel for schedule(static)
    for (int i = 0; i < M; ++i) {
        double *t = (double *)malloc((size_t)R * sizeof(double));
        double *lo = (double *)malloc((size_t)N * sizeof(double));
        double *y = Y + (size_t)i * N;
        row_times_matrix(X + (size_t)i * K, W, y, K, N);
        row_times_matrix(X + (size_t)i * K, A, t, K, R);
        row_times_matrix(t, Bm, lo, R, N);
        for (int n = 0; n < N; ++n) y[n] += alpha * lo[n];
        free(t);
        free(lo);
    }
}
