/*
 * CPU oracle for the Gated MLP   Y = (SiLU(X * W_gate) (.) (X * W_up)) * W_down
 * with an optional RMSNorm prologue on X.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, fp64 statement of what the
 * operator computes.  It is used by the tests, by the smoke check and by the benchmark's
 * CPU-baseline leg; the product (the CUDA library) never links, imports or calls it, and
 * it shares no code, header, table or helper with the CUDA path.
 *
 * What it follows (paper of the Axon superoptimizer):
 *   - the Gated-MLP dataflow graph, figure "mlp-example" (a): matmul(X,W1) -> silu ->
 *     multiply <- matmul(X,W2); matmul(multiply, W3) -> Z.  W1 = gate, W2 = up, W3 = down.
 *   - the granular-operation table of Section 5: matmul(x,y) = sum_k mul(x[i,k], y[k,j]);
 *     silu(x) = mul(x, sigmoid(x)).
 *   - RMSNorm, Eq. (1) of Section 2: X (.) 1/sqrt(mean_i(X_i^2) + eps) along the last
 *     dimension, computed in the graph order square -> mean -> add eps -> rsqrt -> multiply.
 *
 * Readings taken where the paper is silent (the paper is FP32 and proves equivalence over
 * the reals; it fixes no reduced-precision behaviour):
 *   - storage is bf16; every input is widened exactly to fp64 and all arithmetic is fp64;
 *   - the gated product H = silu(G) * U is rounded ONCE to bf16 (round-to-nearest-even),
 *     because that is the one place the GPU data path stores an intermediate (rounding R1);
 *   - with RMSNorm, Xn = x * r * gamma is rounded ONCE to bf16 (rounding R0); gamma is an
 *     optional per-column gain (an extension; gamma == NULL means ones = the paper's form);
 *   - Y is left in fp64 (the reference value the tolerance is taken around);
 *   - every sum runs over its index in ascending order.
 *
 * Pins (tests/test_oracle_*.py): rounding helper against an integer-arithmetic
 * restatement and a library conversion; SiLU identities; RMSNorm unit-RMS / scale
 * invariance; zero-gate, zero-up, zero-down; one-hot closed forms; integer-exact inputs;
 * naive triple-loop matmul from a separate translation unit; torch fp64 cross-check.
 * Not pinned ("parity unpinned"): behaviour on NaN/Inf inputs.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 bits -> double, exact: a bf16 is the upper half of an IEEE binary32. */
double gmlp_oracle_bf16_to_double(uint16_t b)
{
    uint32_t w = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/*
 * double -> bf16 bits, round-to-nearest-even, in ONE rounding (not via binary32).
 * bf16 has 8 significant bits and binary32's exponent range; the spacing of bf16 values
 * around |v| = m * 2^e (m in [0.5,1)) is 2^(e-8), and never finer than 2^-133 (subnormals).
 */
uint16_t gmlp_oracle_bf16_rn(double v)
{
    uint32_t sign = signbit(v) ? 0x8000u : 0u;
    if (isnan(v)) return (uint16_t)(sign | 0x7FC0u);
    if (isinf(v)) return (uint16_t)(sign | 0x7F80u);
    double a = fabs(v);
    if (a == 0.0) return (uint16_t)sign;
    int e;
    (void)frexp(a, &e);
    int q = e - 8;
    if (q < -133) q = -133;
    double r = ldexp(rint(ldexp(a, -q)), q);      /* rint: ties-to-even in the default mode */
    if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80u);
    float f = (float)r;                            /* exact: r is a bf16 value */
    uint32_t w;
    memcpy(&w, &f, sizeof w);
    return (uint16_t)(sign | (w >> 16));
}

/* silu(g) = g * sigmoid(g), written g / (1 + exp(-g)) so that g -> -inf gives -0, not NaN. */
double gmlp_oracle_silu(double g)
{
    return g / (1.0 + exp(-g));
}

/*
 * Gate activation of the gated unit h = act(g) * u.  The paper's Gated MLP uses SiLU; its benchmark list
 * (Section 6.1) also names SwiGLU- and GLU-gated forms without defining them.  Reading taken (the
 * definitions of the GLU-variants literature): kind 0 SiLU g*sigmoid(g); kind 1 Swish-beta
 * g*sigmoid(beta*g) (beta = 1 is SiLU); kind 2 GLU sigmoid(g); kind 3 GELU g*Phi(g), Phi the standard normal
 * distribution function (the exact form, not the tanh approximation), written g * erfc(-g / sqrt 2) / 2 so
 * that the negative tail keeps its relative accuracy.  Anything else: NaN.
 */
double gmlp_oracle_gate_act(double g, int kind, double beta)
{
    switch (kind) {
        case 0: return gmlp_oracle_silu(g);
        case 1: return g / (1.0 + exp(-(beta * g)));
        case 2: return 1.0 / (1.0 + exp(-g));
        case 3: return 0.5 * g * erfc(-g * 0.70710678118654752440);
        default: return NAN;
    }
}

/*
 * RMSNorm of one row (Eq. 1; graph order square, mean, add eps, rsqrt, multiply):
 *   ms = (1/d) sum_k x[k]^2 ;  r = 1/sqrt(ms + eps) ;  xn[k] = bf16_rn(x[k] * r * gamma[k]).
 * Also returns r through *r_out when non-NULL.
 */
void gmlp_oracle_rmsnorm_row(const uint16_t* x, const uint16_t* gamma, float eps,
                             int64_t d_model, uint16_t* xn_out, double* r_out)
{
    double ss = 0.0;
    for (int64_t k = 0; k < d_model; ++k) {
        double v = gmlp_oracle_bf16_to_double(x[k]);
        ss += v * v;
    }
    double ms = ss / (double)d_model;
    double r = 1.0 / sqrt(ms + (double)eps);
    for (int64_t k = 0; k < d_model; ++k) {
        double v = gmlp_oracle_bf16_to_double(x[k]) * r;
        if (gamma) v *= gmlp_oracle_bf16_to_double(gamma[k]);
        xn_out[k] = gmlp_oracle_bf16_rn(v);
    }
    if (r_out) *r_out = r;
}

/*
 * The operator on a list of rows.  All matrices are dense row-major bf16 bit patterns:
 *   X [M, d_model], Wg/Wu [d_model, d_ff], Wd [d_ff, d_model], gamma [d_model] or NULL.
 * rows[0..n_rows) selects the rows of X to compute (rows are independent of each other).
 * Outputs: Y_ref [n_rows, d_model] fp64 (not rounded); H_bits [n_rows, d_ff] bf16 bits
 * (may be NULL); Xn_bits [n_rows, d_model] (may be NULL; the row as fed to the matmuls).
 * Returns 0, or -1 on a bad argument / allocation failure.
 */
int gmlp_oracle_rows_act(const uint16_t* X, const uint16_t* Wg, const uint16_t* Wu, const uint16_t* Wd,
                         const uint16_t* gamma, float eps, int rmsnorm,
                         int64_t M, int64_t d_model, int64_t d_ff,
                         const int64_t* rows, int64_t n_rows,
                         double* Y_ref, uint16_t* H_bits, uint16_t* Xn_bits, int num_threads,
                         int act_kind, double act_beta)
{
    if (!X || !Wg || !Wu || !Wd || !rows || !Y_ref || M < 0 || d_model <= 0 || d_ff <= 0 || n_rows < 0)
        return -1;
    for (int64_t i = 0; i < n_rows; ++i)
        if (rows[i] < 0 || rows[i] >= M) return -1;
    int failed = 0;
#ifdef _OPENMP
    omp_set_num_threads(num_threads > 0 ? num_threads : omp_get_num_procs());   /* 0 = all cores, whatever an earlier call asked for */
#else
    (void)num_threads;
#endif
#pragma omp parallel
    {
        double* xn = (double*)malloc(sizeof(double) * (size_t)d_model);
        uint16_t* xnb = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)d_model);
        double* g = (double*)malloc(sizeof(double) * (size_t)d_ff);
        double* u = (double*)malloc(sizeof(double) * (size_t)d_ff);
        double* h = (double*)malloc(sizeof(double) * (size_t)d_ff);
        if (!xn || !xnb || !g || !u || !h) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int64_t i = 0; i < n_rows; ++i) {
                const uint16_t* x = X + rows[i] * d_model;
                /* a0: optional RMSNorm prologue, rounding R0 */
                if (rmsnorm) {
                    gmlp_oracle_rmsnorm_row(x, gamma, eps, d_model, xnb, NULL);
                } else {
                    memcpy(xnb, x, sizeof(uint16_t) * (size_t)d_model);
                }
                for (int64_t k = 0; k < d_model; ++k) xn[k] = gmlp_oracle_bf16_to_double(xnb[k]);
                if (Xn_bits) memcpy(Xn_bits + i * d_model, xnb, sizeof(uint16_t) * (size_t)d_model);
                /* a1, a2: G = xn * Wg, U = xn * Wu; each g[n], u[n] sums k = 0, 1, 2, ... */
                for (int64_t n = 0; n < d_ff; ++n) { g[n] = 0.0; u[n] = 0.0; }
                for (int64_t k = 0; k < d_model; ++k) {
                    const double xk = xn[k];
                    const uint16_t* wg = Wg + k * d_ff;
                    const uint16_t* wu = Wu + k * d_ff;
                    for (int64_t n = 0; n < d_ff; ++n) {
                        g[n] += xk * gmlp_oracle_bf16_to_double(wg[n]);
                        u[n] += xk * gmlp_oracle_bf16_to_double(wu[n]);
                    }
                }
                /* a3, a4: H = bf16_rn(silu(G) * U), rounding R1 */
                for (int64_t n = 0; n < d_ff; ++n) {
                    uint16_t hb = gmlp_oracle_bf16_rn(gmlp_oracle_gate_act(g[n], act_kind, act_beta) * u[n]);
                    if (H_bits) H_bits[i * d_ff + n] = hb;
                    h[n] = gmlp_oracle_bf16_to_double(hb);
                }
                /* a5: Y = H * Wd; each y[c] sums n = 0, 1, 2, ... ; not rounded */
                double* y = Y_ref + i * d_model;
                for (int64_t c = 0; c < d_model; ++c) y[c] = 0.0;
                for (int64_t n = 0; n < d_ff; ++n) {
                    const double hn = h[n];
                    const uint16_t* wd = Wd + n * d_model;
                    for (int64_t c = 0; c < d_model; ++c)
                        y[c] += hn * gmlp_oracle_bf16_to_double(wd[c]);
                }
            }
        }
        free(xn); free(xnb); free(g); free(u); free(h);
    }
    return failed ? -1 : 0;
}

/* The operator as the paper states it: SiLU gate. */
int gmlp_oracle_rows(const uint16_t* X, const uint16_t* Wg, const uint16_t* Wu, const uint16_t* Wd,
                     const uint16_t* gamma, float eps, int rmsnorm,
                     int64_t M, int64_t d_model, int64_t d_ff,
                     const int64_t* rows, int64_t n_rows,
                     double* Y_ref, uint16_t* H_bits, uint16_t* Xn_bits, int num_threads)
{
    return gmlp_oracle_rows_act(X, Wg, Wu, Wd, gamma, eps, rmsnorm, M, d_model, d_ff, rows, n_rows,
                                Y_ref, H_bits, Xn_bits, num_threads, 0, 1.0);
}

/*
 * The gate/up half on its own ("Matmul+Matmul+SiLU+Mul" of the paper's benchmark list, Section 6.1):
 *   P[i, n] = silu(sum_k xn[k] Wg[k, n]) * (sum_k xn[k] Wu[k, n])      for the selected rows,
 * returned in fp64 WITHOUT the final rounding (the GPU rounds P once to bf16; the tolerance is taken
 * around this value).  Same conventions as gmlp_oracle_rows; the optional RMSNorm prologue rounds Xn.
 */
int gmlp_oracle_gate_up_rows_act(const uint16_t* X, const uint16_t* Wg, const uint16_t* Wu,
                                 const uint16_t* gamma, float eps, int rmsnorm,
                                 int64_t M, int64_t d_model, int64_t d_ff,
                                 const int64_t* rows, int64_t n_rows, double* P, int num_threads,
                                 int act_kind, double act_beta)
{
    if (!X || !Wg || !Wu || !rows || !P || M < 0 || d_model <= 0 || d_ff <= 0 || n_rows < 0) return -1;
    for (int64_t i = 0; i < n_rows; ++i)
        if (rows[i] < 0 || rows[i] >= M) return -1;
    int failed = 0;
#ifdef _OPENMP
    omp_set_num_threads(num_threads > 0 ? num_threads : omp_get_num_procs());   /* 0 = all cores, whatever an earlier call asked for */
#else
    (void)num_threads;
#endif
#pragma omp parallel
    {
        double* xn = (double*)malloc(sizeof(double) * (size_t)d_model);
        uint16_t* xnb = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)d_model);
        double* g = (double*)malloc(sizeof(double) * (size_t)d_ff);
        double* u = (double*)malloc(sizeof(double) * (size_t)d_ff);
        if (!xn || !xnb || !g || !u) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int64_t i = 0; i < n_rows; ++i) {
                const uint16_t* x = X + rows[i] * d_model;
                if (rmsnorm) gmlp_oracle_rmsnorm_row(x, gamma, eps, d_model, xnb, NULL);
                else memcpy(xnb, x, sizeof(uint16_t) * (size_t)d_model);
                for (int64_t k = 0; k < d_model; ++k) xn[k] = gmlp_oracle_bf16_to_double(xnb[k]);
                for (int64_t n = 0; n < d_ff; ++n) { g[n] = 0.0; u[n] = 0.0; }
                for (int64_t k = 0; k < d_model; ++k) {
                    const double xk = xn[k];
                    const uint16_t* wg = Wg + k * d_ff;
                    const uint16_t* wu = Wu + k * d_ff;
                    for (int64_t n = 0; n < d_ff; ++n) {
                        g[n] += xk * gmlp_oracle_bf16_to_double(wg[n]);
                        u[n] += xk * gmlp_oracle_bf16_to_double(wu[n]);
                    }
                }
                for (int64_t n = 0; n < d_ff; ++n) P[i * d_ff + n] = gmlp_oracle_gate_act(g[n], act_kind, act_beta) * u[n];
            }
        }
        free(xn); free(xnb); free(g); free(u);
    }
    return failed ? -1 : 0;
}

int gmlp_oracle_gate_up_rows(const uint16_t* X, const uint16_t* Wg, const uint16_t* Wu,
                             const uint16_t* gamma, float eps, int rmsnorm,
                             int64_t M, int64_t d_model, int64_t d_ff,
                             const int64_t* rows, int64_t n_rows, double* P, int num_threads)
{
    return gmlp_oracle_gate_up_rows_act(X, Wg, Wu, gamma, eps, rmsnorm, M, d_model, d_ff, rows, n_rows, P,
                                        num_threads, 0, 1.0);
}

/*
 * RMSNorm followed by a matrix multiplication, the paper's running example (Section 2, Eq. 1 and
 * figure "rmsnorm-matmul-comp-graph" (a)):   Z = RMSNorm(X) * W,
 *   r_i = 1/sqrt(mean_k X[i,k]^2 + eps),   Z[i, n] = sum_k (X[i,k] * r_i * gamma[k]) * W[k, n].
 * Plain definition in fp64 with no intermediate rounding; gamma == NULL is the paper's gain-less form.
 * X [M, K], W [K, N] bf16 bit patterns; Z [n_rows, N] fp64 for the selected rows.
 */
int gmlp_oracle_rmsnorm_matmul_rows(const uint16_t* X, const uint16_t* W, const uint16_t* gamma, float eps,
                                    int64_t M, int64_t K, int64_t N, const int64_t* rows, int64_t n_rows,
                                    double* Z, int num_threads)
{
    if (!X || !W || !rows || !Z || M < 0 || K <= 0 || N <= 0 || n_rows < 0) return -1;
    for (int64_t i = 0; i < n_rows; ++i)
        if (rows[i] < 0 || rows[i] >= M) return -1;
    int failed = 0;
#ifdef _OPENMP
    omp_set_num_threads(num_threads > 0 ? num_threads : omp_get_num_procs());   /* 0 = all cores, whatever an earlier call asked for */
#else
    (void)num_threads;
#endif
#pragma omp parallel
    {
        double* xn = (double*)malloc(sizeof(double) * (size_t)K);
        if (!xn) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int64_t i = 0; i < n_rows; ++i) {
                const uint16_t* x = X + rows[i] * K;
                double ss = 0.0;
                for (int64_t k = 0; k < K; ++k) {
                    const double v = gmlp_oracle_bf16_to_double(x[k]);
                    ss += v * v;
                }
                const double r = 1.0 / sqrt(ss / (double)K + (double)eps);
                for (int64_t k = 0; k < K; ++k) {
                    double v = gmlp_oracle_bf16_to_double(x[k]) * r;
                    if (gamma) v *= gmlp_oracle_bf16_to_double(gamma[k]);
                    xn[k] = v;
                }
                double* z = Z + i * N;
                for (int64_t n = 0; n < N; ++n) z[n] = 0.0;
                for (int64_t k = 0; k < K; ++k) {
                    const double xk = xn[k];
                    const uint16_t* w = W + k * N;
                    for (int64_t n = 0; n < N; ++n) z[n] += xk * gmlp_oracle_bf16_to_double(w[n]);
                }
            }
        }
        free(xn);
    }
    return failed ? -1 : 0;
}

/*
 * A matrix multiplication, a residual addition and RMSNorm ("Matmul+Add+RMSNorm" of the paper's
 * benchmark list, Section 6.1; the paper names the chain and does not spell out the graph):
 *     S = X * W + R,     Z = RMSNorm(S)      (Eq. 1 along the last dimension, N)
 * Readings taken: S is an output as well (the updated residual stream), stored in bf16 with ONE
 * rounding of the fp64 sum; the RMSNorm is the one of Eq. (1) applied to the STORED S (what a
 * following operator would read), in fp64, with the optional per-column gain gamma [N]; Z is left in
 * fp64 (the value the tolerance is taken around).
 * X [M, K], W [K, N], R [M, N], gamma [N] or NULL: bf16 bit patterns.  For the selected rows:
 * S_bits [n_rows, N] bf16 bits (may be NULL), S_ref [n_rows, N] fp64 unrounded sums (may be NULL),
 * Z [n_rows, N] fp64.
 */
int gmlp_oracle_matmul_add_rmsnorm_rows(const uint16_t* X, const uint16_t* W, const uint16_t* R,
                                        const uint16_t* gamma, float eps, int64_t M, int64_t K, int64_t N,
                                        const int64_t* rows, int64_t n_rows,
                                        uint16_t* S_bits, double* S_ref, double* Z, int num_threads)
{
    if (!X || !W || !R || !rows || !Z || M < 0 || K <= 0 || N <= 0 || n_rows < 0) return -1;
    for (int64_t i = 0; i < n_rows; ++i)
        if (rows[i] < 0 || rows[i] >= M) return -1;
    int failed = 0;
#ifdef _OPENMP
    omp_set_num_threads(num_threads > 0 ? num_threads : omp_get_num_procs());   /* 0 = all cores, whatever an earlier call asked for */
#else
    (void)num_threads;
#endif
#pragma omp parallel
    {
        double* s = (double*)malloc(sizeof(double) * (size_t)N);
        if (!s) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int64_t i = 0; i < n_rows; ++i) {
                const uint16_t* x = X + rows[i] * K;
                const uint16_t* res = R + rows[i] * N;
                for (int64_t n = 0; n < N; ++n) s[n] = 0.0;
                for (int64_t k = 0; k < K; ++k) {
                    const double xk = gmlp_oracle_bf16_to_double(x[k]);
                    const uint16_t* w = W + k * N;
                    for (int64_t n = 0; n < N; ++n) s[n] += xk * gmlp_oracle_bf16_to_double(w[n]);
                }
                double ss = 0.0;
                for (int64_t n = 0; n < N; ++n) {
                    s[n] += gmlp_oracle_bf16_to_double(res[n]);
                    if (S_ref) S_ref[i * N + n] = s[n];
                    const uint16_t sb = gmlp_oracle_bf16_rn(s[n]);
                    if (S_bits) S_bits[i * N + n] = sb;
                    s[n] = gmlp_oracle_bf16_to_double(sb);
                    ss += s[n] * s[n];
                }
                const double r = 1.0 / sqrt(ss / (double)N + (double)eps);
                for (int64_t n = 0; n < N; ++n) {
                    double v = s[n] * r;
                    if (gamma) v *= gmlp_oracle_bf16_to_double(gamma[n]);
                    Z[i * N + n] = v;
                }
            }
        }
        free(s);
    }
    return failed ? -1 : 0;
}

/*
 * A plain matrix multiplication on selected rows, Z[i, n] = sum_k X[rows[i], k] * W[k, n] in fp64 (the granular
 * definition of matmul in Section 5's operation table).  It is the reference for each of the three products of
 * the QKV projection (Section 6.1), which share X and nothing else.  X [M, K], W [K, N] bf16 bit patterns.
 */
int gmlp_oracle_matmul_rows(const uint16_t* X, const uint16_t* W, int64_t M, int64_t K, int64_t N,
                            const int64_t* rows, int64_t n_rows, double* Z, int num_threads)
{
    if (!X || !W || !rows || !Z || M < 0 || K <= 0 || N <= 0 || n_rows < 0) return -1;
    for (int64_t i = 0; i < n_rows; ++i)
        if (rows[i] < 0 || rows[i] >= M) return -1;
#ifdef _OPENMP
    omp_set_num_threads(num_threads > 0 ? num_threads : omp_get_num_procs());   /* 0 = all cores, whatever an earlier call asked for */
#else
    (void)num_threads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n_rows; ++i) {
        const uint16_t* x = X + rows[i] * K;
        double* z = Z + i * N;
        for (int64_t n = 0; n < N; ++n) z[n] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            const double xk = gmlp_oracle_bf16_to_double(x[k]);
            const uint16_t* w = W + k * N;
            for (int64_t n = 0; n < N; ++n) z[n] += xk * gmlp_oracle_bf16_to_double(w[n]);
        }
    }
    return 0;
}

/*
 * Group Query Attention (one of the paper's multi-operator kernels, Section 6.1; the paper names it and gives no
 * graph).  Reading taken - the standard definition, no mask:
 *     for query head h (0 <= h < Hq), with key/value head g = h / (Hq / Hkv):
 *         P = softmax_s( Q_h K_g^T / sqrt(D) ),      O_h = P V_g
 * Q [M, Hq*D], K and V [S, Hkv*D], O [M, Hq*D] row-major (head h occupies columns [h*D, (h+1)*D)); bf16 bit
 * patterns in, everything in fp64, softmax written out as max-subtracted exponentials over their sum, O left in
 * fp64.  For the selected query rows: O_ref [n_rows, Hq*D].
 * causal != 0 (an extension; decoder models use it): query row m sees keys s <= m + (S - M) only, i.e. the
 * queries are the LAST M positions of the S-long sequence (needs S >= M); masked scores take no part in the
 * softmax.
 */
int gmlp_oracle_gqa_rows(const uint16_t* Q, const uint16_t* K, const uint16_t* V, int64_t M, int64_t S,
                         int64_t Hq, int64_t Hkv, int64_t D, const int64_t* rows, int64_t n_rows,
                         double* O_ref, int num_threads, int causal)
{
    if (!Q || !K || !V || !rows || !O_ref || M < 0 || S <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || n_rows < 0) return -1;
    if (Hq % Hkv != 0) return -1;
    if (causal && S < M) return -1;
    for (int64_t i = 0; i < n_rows; ++i)
        if (rows[i] < 0 || rows[i] >= M) return -1;
    const int64_t group = Hq / Hkv;
    const double scale = 1.0 / sqrt((double)D);
    int failed = 0;
#ifdef _OPENMP
    omp_set_num_threads(num_threads > 0 ? num_threads : omp_get_num_procs());   /* 0 = all cores, whatever an earlier call asked for */
#else
    (void)num_threads;
#endif
#pragma omp parallel
    {
        double* p = (double*)malloc(sizeof(double) * (size_t)S);
        if (!p) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for collapse(2) schedule(dynamic, 1)
            for (int64_t i = 0; i < n_rows; ++i) {
                for (int64_t h = 0; h < Hq; ++h) {
                    const uint16_t* q = Q + rows[i] * Hq * D + h * D;
                    const int64_t g = h / group;
                    const int64_t S_vis = causal ? rows[i] + (S - M) + 1 : S;      /* keys this row may see */
                    double mx = -INFINITY;
                    for (int64_t s = 0; s < S_vis; ++s) {
                        const uint16_t* k = K + s * Hkv * D + g * D;
                        double dot = 0.0;
                        for (int64_t d = 0; d < D; ++d) dot += gmlp_oracle_bf16_to_double(q[d]) * gmlp_oracle_bf16_to_double(k[d]);
                        p[s] = dot * scale;
                        if (p[s] > mx) mx = p[s];
                    }
                    double sum = 0.0;
                    for (int64_t s = 0; s < S_vis; ++s) {
                        p[s] = exp(p[s] - mx);
                        sum += p[s];
                    }
                    double* o = O_ref + i * Hq * D + h * D;
                    for (int64_t d = 0; d < D; ++d) o[d] = 0.0;
                    for (int64_t s = 0; s < S_vis; ++s) {
                        const double w = p[s] / sum;
                        const uint16_t* v = V + s * Hkv * D + g * D;
                        for (int64_t d = 0; d < D; ++d) o[d] += w * gmlp_oracle_bf16_to_double(v[d]);
                    }
                }
            }
        }
        free(p);
    }
    return failed ? -1 : 0;
}

/* Array forms of the two scalar helpers (plain loops), for the tests. */
void gmlp_oracle_bf16_rn_array(const double* v, uint16_t* out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = gmlp_oracle_bf16_rn(v[i]);
}

void gmlp_oracle_gate_act_array(const double* v, double* out, int64_t n, int kind, double beta)
{
    for (int64_t i = 0; i < n; ++i) out[i] = gmlp_oracle_gate_act(v[i], kind, beta);
}

void gmlp_oracle_silu_array(const double* v, double* out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = gmlp_oracle_silu(v[i]);
}

/* Threads the parallel region above will use (for the benchmark's "cores" field). */
int gmlp_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
