/*
 * CPU oracle for the inference-time Mixture-of-Lookup-Experts (MoLE) layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the layer
 * computes, evaluated in fp64.  It shares no code with the CUDA library and is never on
 * the product path: only the tests, the smoke check and the bench's CPU-baseline leg
 * execute it.
 *
 * Every function follows one passage of the paper (arXiv 2503.15798):
 *   oracle_gelu / oracle_ffn      the routed expert FFN_j of Sec. 3.2 (two matrices, no
 *                                 bias: Table 1 counts 2*d*D parameters and 4*d*D FLOPs)
 *   oracle_rmsnorm                the expert_layernorm of the training listing (App. A.1)
 *   oracle_build_lut              Eq. 6 and Eq. 7: v^i_j = FFN_j(Embedding(i)) for every id
 *   oracle_router_gates           Eq. 4: softmax over ALL N router logits h . r_j
 *   oracle_layer_lookup           Eq. 8 without the shared expert: h' = sum_j g_j v^i_j + h
 *   oracle_layer_onthefly         Eq. 5 without the shared expert: h' = sum_j g_j FFN_j(e) + h
 *   oracle_dedup                  unique ids of one step (the offload mode's first step)
 *
 * Readings taken where the paper is silent or garbled:
 *   - FFN_j(x) = W2 . gelu(W1 . x), exact (erf) GELU, no bias, not gated.
 *   - the weighted sum runs over the expert axis (Eq. 8); the inference listing's
 *     "sum(dim=2)" on a 3-D tensor is a typo for the expert axis.
 *   - router weight is row-major [d][N] (logits = hidden @ W_r), no bias, no temperature.
 *   - the table is row-major [V][N][d].
 *   - position t uses its own input id ids[t]; tokens are independent.
 *   - an id outside [0, V) contributes no routed term (out = residual) and is counted in
 *     the return value.
 *
 * Pins (tests/test_oracle_*.py): erf-GELU against the normal CDF, a hand-worked FFN, a
 * worked layer example with rational gates (logits ln 3 and 0), W_r = 0 => mean of the
 * rows, N = 1, exact one-hot gather, lookup form == on-the-fly form (Eq. 5 with Eq. 6
 * substituted == Eq. 8), the library routines torch.nn.functional.embedding_bag /
 * scipy softmax / numpy matmul on the special cases they cover, and the parameter counts
 * printed in Tables 3, 6 and 8.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC oracle/mole_oracle.c -o oracle/libmole_oracle.so -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_F64 0
#define ORACLE_F32 1
#define ORACLE_BF16 2

/* Widen element `i` of an array of the given storage type to double, exactly. */
static double widen(const void *p, int64_t i, int dtype)
{
    if (dtype == ORACLE_F64) return ((const double *)p)[i];
    if (dtype == ORACLE_F32) return (double)((const float *)p)[i];
    /* bf16: the upper 16 bits of an IEEE binary32 */
    uint32_t bits = ((uint32_t)((const uint16_t *)p)[i]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* Exact GELU: x * Phi(x), Phi the standard normal CDF. */
double oracle_gelu(double x)
{
    return 0.5 * x * (1.0 + erf(x / sqrt(2.0)));
}

/* y = W2 . gelu(W1 . x);  W1 is [D][d], W2 is [d][D], both row-major. */
void oracle_ffn(const double *x, const double *W1, const double *W2, int d, int D, double *y)
{
    double *a = (double *)malloc(sizeof(double) * (size_t)D);
    for (int k = 0; k < D; ++k) {
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += W1[(size_t)k * d + c] * x[c];
        a[k] = oracle_gelu(s);
    }
    for (int c = 0; c < d; ++c) {
        double s = 0.0;
        for (int k = 0; k < D; ++k) s += W2[(size_t)c * D + k] * a[k];
        y[c] = s;
    }
    free(a);
}

/* y = x / sqrt(mean(x^2) + eps) * w */
void oracle_rmsnorm(const double *x, const double *w, double eps, int d, double *y)
{
    double ms = 0.0;
    for (int c = 0; c < d; ++c) ms += x[c] * x[c];
    ms /= (double)d;
    double r = 1.0 / sqrt(ms + eps);
    for (int c = 0; c < d; ++c) y[c] = x[c] * r * w[c];
}

/*
 * Eq. 6 / Eq. 7: lut[i][j][:] = FFN_j(E[i]) for every id i and expert j.
 * E [V][d]; W1 [N][D][d]; W2 [N][d][D]; lut [V][N][d].  If norm_w is not NULL the
 * embedding row first goes through RMSNorm(norm_w, eps), as the training listing does.
 */
void oracle_build_lut(const double *E, const double *W1, const double *W2, const double *norm_w,
                      double eps, int V, int d, int D, int N, double *lut)
{
    double *e = (double *)malloc(sizeof(double) * (size_t)d);
    for (int i = 0; i < V; ++i) {
        if (norm_w) oracle_rmsnorm(E + (size_t)i * d, norm_w, eps, d, e);
        else memcpy(e, E + (size_t)i * d, sizeof(double) * (size_t)d);
        for (int j = 0; j < N; ++j)
            oracle_ffn(e, W1 + (size_t)j * D * d, W2 + (size_t)j * d * D, d, D,
                       lut + ((size_t)i * N + j) * d);
    }
    free(e);
}

/* Eq. 4: g = softmax(z), z_j = sum_c h[c] * Wr[c][j].  Wr is [d][N]. */
void oracle_router_gates(const double *h, const double *Wr, int d, int N, double *g)
{
    double zmax = -INFINITY;
    for (int j = 0; j < N; ++j) {
        double z = 0.0;
        for (int c = 0; c < d; ++c) z += h[c] * Wr[(size_t)c * N + j];
        g[j] = z;
        if (z > zmax) zmax = z;
    }
    double sum = 0.0;
    for (int j = 0; j < N; ++j) {
        g[j] = exp(g[j] - zmax);
        sum += g[j];
    }
    for (int j = 0; j < N; ++j) g[j] /= sum;
}

/*
 * Eq. 8 (lookup form, shared expert left to the caller):
 *   out[t][c] = res[t][c] + sum_j g_j(hidden[t]) * lut[ids[t]][j][c]
 * hidden/residual [M][d], lut [V][N][d], w_router [d][N] are stored as `dtype`
 * (ORACLE_F64 / ORACLE_F32 / ORACLE_BF16) and widened exactly; residual == NULL means
 * residual = hidden.  out [M][d] and gates [M][N] (may be NULL) are fp64 and unrounded.
 * `threads` > 1 splits the token loop across OpenMP threads (tokens are independent).
 * Returns the number of ids outside [0, V).
 */
int64_t oracle_layer_lookup(const void *hidden, const int64_t *ids, const void *lut,
                            const void *w_router, const void *residual, int dtype, int64_t M,
                            int N, int d, int64_t V, double *out, double *gates, int threads)
{
    int64_t bad = 0;
    double *Wr = (double *)malloc(sizeof(double) * (size_t)d * N);
    for (int64_t k = 0; k < (int64_t)d * N; ++k) Wr[k] = widen(w_router, k, dtype);
    if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) reduction(+ : bad) schedule(static)
    for (int64_t t = 0; t < M; ++t) {
        double *h = (double *)malloc(sizeof(double) * (size_t)d);
        double *g = (double *)malloc(sizeof(double) * (size_t)N);
        for (int c = 0; c < d; ++c) h[c] = widen(hidden, t * d + c, dtype);
        oracle_router_gates(h, Wr, d, N, g);
        if (gates)
            for (int j = 0; j < N; ++j) gates[t * N + j] = g[j];
        int64_t id = ids[t];
        int ok = (id >= 0 && id < V);
        if (!ok) bad += 1;
        for (int c = 0; c < d; ++c) {
            double s = 0.0;
            if (ok)
                for (int j = 0; j < N; ++j)
                    s += g[j] * widen(lut, (id * N + j) * (int64_t)d + c, dtype);
            double r = residual ? widen(residual, t * d + c, dtype) : h[c];
            out[t * d + c] = r + s;
        }
        free(h);
        free(g);
    }
    free(Wr);
    return bad;
}

/*
 * Eq. 5 (training-time / on-the-fly form, shared expert left to the caller):
 *   out[t] = hidden[t] + sum_j g_j(hidden[t]) * FFN_j(E[ids[t]])
 * All arrays fp64: hidden [M][d], E [V][d], W1 [N][D][d], W2 [N][d][D], Wr [d][N].
 * norm_w (or NULL) as in oracle_build_lut.
 */
int64_t oracle_layer_onthefly(const double *hidden, const int64_t *ids, const double *E,
                              const double *W1, const double *W2, const double *Wr,
                              const double *norm_w, double eps, int64_t M, int N, int d, int D,
                              int64_t V, double *out)
{
    int64_t bad = 0;
    double *g = (double *)malloc(sizeof(double) * (size_t)N);
    double *e = (double *)malloc(sizeof(double) * (size_t)d);
    double *y = (double *)malloc(sizeof(double) * (size_t)d);
    for (int64_t t = 0; t < M; ++t) {
        const double *h = hidden + t * d;
        oracle_router_gates(h, Wr, d, N, g);
        for (int c = 0; c < d; ++c) out[t * d + c] = h[c];
        int64_t id = ids[t];
        if (id < 0 || id >= V) {
            bad += 1;
            continue;
        }
        if (norm_w) oracle_rmsnorm(E + id * d, norm_w, eps, d, e);
        else memcpy(e, E + id * d, sizeof(double) * (size_t)d);
        for (int j = 0; j < N; ++j) {
            oracle_ffn(e, W1 + (size_t)j * D * d, W2 + (size_t)j * d * D, d, D, y);
            for (int c = 0; c < d; ++c) out[t * d + c] += g[j] * y[c];
        }
    }
    free(g);
    free(e);
    free(y);
    return bad;
}

/*
 * Unique ids of a step, in order of first occurrence, by the plain quadratic definition:
 * uniq[0..U) are the distinct values of ids, slot[t] is the position with
 * uniq[slot[t]] == ids[t].  Returns U.
 */
int64_t oracle_dedup(const int64_t *ids, int64_t M, int64_t *uniq, int64_t *slot)
{
    int64_t U = 0;
    for (int64_t t = 0; t < M; ++t) {
        int64_t u = 0;
        while (u < U && uniq[u] != ids[t]) ++u;
        if (u == U) uniq[U++] = ids[t];
        slot[t] = u;
    }
    return U;
}

/* Threads an OpenMP region of `threads` would really get on this machine. */
int oracle_effective_threads(int threads)
{
    int n = 1;
#ifdef _OPENMP
    if (threads < 1) threads = 1;
#pragma omp parallel num_threads(threads)
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#else
    (void)threads;
#endif
    return n;
}
