/*
 * CPU oracle for the Monarch multiply (Dao et al., arXiv 2204.00595).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain fp64 statement of
 * what the hot path computes.  It shares nothing with the CUDA library: no
 * header, no helper, no table.  Only tests, the smoke check and the CPU
 * baseline leg of the benchmark may call it.
 *
 * Notation (0-indexed; the paper's Section 3.3 uses 1-indexed subscripts):
 *   n = m*m                                   (Definition 3.1)
 *   x[t][k*m + i]    token t, viewed as an m x m matrix x_{ki}
 *   R[k][j][i]       block k of R, output row j, input column i
 *   L[j][l][k]       block j of L, output row l, input column k
 *   u[t][k][j]       the paper's intermediate "y_{kj}" of step 1
 *   y[t][l*m + j]    the paper's "z_{lj}" of steps 2-3, flattened l-major
 *
 * Every loop nest below is the formula of the cited passage written out;
 * there is no blocking, fusion or reordering.  OpenMP only distributes
 * independent tokens (or independent weight blocks) over host cores.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Step 1 of the multiply (Section 3.3, "Steps to multiply x by a Monarch
 * matrix", item 1):  u_{kj} = sum_i R_{kji} x_{ki}. */
static void step1_one_token(const double *x, const double *R, double *u, int m)
{
    for (int k = 0; k < m; ++k)
        for (int j = 0; j < m; ++j) {
            double acc = 0.0;
            for (int i = 0; i < m; ++i)
                acc += R[((size_t)k * m + j) * m + i] * x[(size_t)k * m + i];
            u[(size_t)k * m + j] = acc;
        }
}

/* Steps 2-3 (same passage, items 2 and 3):  z_{lj} = sum_k L_{jlk} u_{kj},
 * returned flattened with l major and j minor. */
static void step23_one_token(const double *u, const double *L, double *y, int m)
{
    for (int l = 0; l < m; ++l)
        for (int j = 0; j < m; ++j) {
            double acc = 0.0;
            for (int k = 0; k < m; ++k)
                acc += L[((size_t)j * m + l) * m + k] * u[(size_t)k * m + j];
            y[(size_t)l * m + j] = acc;
        }
}

/* y = M x for T tokens; u_out (T*n doubles) may be NULL. */
int oracle_fwd(const double *x, const double *L, const double *R, double *y,
               double *u_out, long T, int m)
{
    const size_t n = (size_t)m * m;
    int fail = 0;
#pragma omp parallel
    {
        double *u = (double *)malloc(n * sizeof(double));
        if (!u) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(static)
            for (long t = 0; t < T; ++t) {
                step1_one_token(x + (size_t)t * n, R, u, m);
                step23_one_token(u, L, y + (size_t)t * n, m);
                if (u_out) memcpy(u_out + (size_t)t * n, u, n * sizeof(double));
            }
        }
        free(u);
    }
    return fail;
}

/* Dense materialisation by the entry formula, Eq. (2):
 *   M_{l j k i} = L_{j l k} R_{k j i},  row index l*m+j, column index k*m+i
 * (the index map of Algorithm 1's reshape). Mdense is n x n row-major. */
void oracle_dense(const double *L, const double *R, double *Mdense, int m)
{
    const size_t n = (size_t)m * m;
    for (int l = 0; l < m; ++l)
        for (int j = 0; j < m; ++j)
            for (int k = 0; k < m; ++k)
                for (int i = 0; i < m; ++i)
                    Mdense[((size_t)l * m + j) * n + (size_t)k * m + i] =
                        L[((size_t)j * m + l) * m + k] * R[((size_t)k * m + j) * m + i];
}

/* Gradients of  f = <dy, M x>  (the paper trains by automatic
 * differentiation, Section 4; these are the adjoints of steps 1-3):
 *   du[t][k][j] = sum_l L[j][l][k] dy[t][l*m+j]
 *   dx[t][k*m+i] = sum_j R[k][j][i] du[t][k][j]
 *   dL[j][l][k] = sum_t dy[t][l*m+j] u[t][k][j]
 *   dR[k][j][i] = sum_t du[t][k][j] x[t][k*m+i]
 * Any of dx, dL, dR may be NULL.  dL and dR are overwritten. */
int oracle_bwd(const double *x, const double *dy, const double *L, const double *R,
               double *dx, double *dL, double *dR, long T, int m)
{
    const size_t n = (size_t)m * m;
    double *u = (double *)malloc((size_t)T * n * sizeof(double));
    double *du = (double *)malloc((size_t)T * n * sizeof(double));
    if (!u || !du) {
        free(u);
        free(du);
        return 1;
    }
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        const double *xt = x + (size_t)t * n;
        const double *dyt = dy + (size_t)t * n;
        double *ut = u + (size_t)t * n;
        double *dut = du + (size_t)t * n;
        step1_one_token(xt, R, ut, m);
        for (int k = 0; k < m; ++k)
            for (int j = 0; j < m; ++j) {
                double acc = 0.0;
                for (int l = 0; l < m; ++l)
                    acc += L[((size_t)j * m + l) * m + k] * dyt[(size_t)l * m + j];
                dut[(size_t)k * m + j] = acc;
            }
        if (dx) {
            double *dxt = dx + (size_t)t * n;
            for (int k = 0; k < m; ++k)
                for (int i = 0; i < m; ++i) {
                    double acc = 0.0;
                    for (int j = 0; j < m; ++j)
                        acc += R[((size_t)k * m + j) * m + i] * dut[(size_t)k * m + j];
                    dxt[(size_t)k * m + i] = acc;
                }
        }
    }
    if (dL) {
#pragma omp parallel for schedule(static)
        for (int j = 0; j < m; ++j)
            for (int l = 0; l < m; ++l)
                for (int k = 0; k < m; ++k) {
                    double acc = 0.0;
                    for (long t = 0; t < T; ++t)
                        acc += dy[(size_t)t * n + (size_t)l * m + j] *
                               u[(size_t)t * n + (size_t)k * m + j];
                    dL[((size_t)j * m + l) * m + k] = acc;
                }
    }
    if (dR) {
#pragma omp parallel for schedule(static)
        for (int k = 0; k < m; ++k)
            for (int j = 0; j < m; ++j)
                for (int i = 0; i < m; ++i) {
                    double acc = 0.0;
                    for (long t = 0; t < T; ++t)
                        acc += du[(size_t)t * n + (size_t)k * m + j] *
                               x[(size_t)t * n + (size_t)k * m + i];
                    dR[((size_t)k * m + j) * m + i] = acc;
                }
    }
    free(u);
    free(du);
    return 0;
}

/* Monarch feed-forward block: the paper replaces the FFN weight matrices by
 * Monarch matrices (Section 4, end-to-end setting); the block evaluated is
 *   h = GELU(M1 x + b1),  y = M2 h + b2,  GELU(a) = a/2 (1 + erf(a/sqrt 2)). */
int oracle_mlp_fwd(const double *x, const double *L1, const double *R1, const double *b1,
                   const double *L2, const double *R2, const double *b2, double *y,
                   long T, int m)
{
    const size_t n = (size_t)m * m;
    int fail = 0;
#pragma omp parallel
    {
        double *u = (double *)malloc(n * sizeof(double));
        double *h = (double *)malloc(n * sizeof(double));
        if (!u || !h) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(static)
            for (long t = 0; t < T; ++t) {
                step1_one_token(x + (size_t)t * n, R1, u, m);
                step23_one_token(u, L1, h, m);
                for (size_t q = 0; q < n; ++q) {
                    const double a = h[q] + b1[q];
                    h[q] = 0.5 * a * (1.0 + erf(a / sqrt(2.0)));
                }
                step1_one_token(h, R2, u, m);
                double *yt = y + (size_t)t * n;
                step23_one_token(u, L2, yt, m);
                for (size_t q = 0; q < n; ++q) yt[q] += b2[q];
            }
        }
        free(u);
        free(h);
    }
    return fail;
}

/* Gradients of  f = <dy, y>  for the feed-forward block above (the paper
 * trains it by automatic differentiation, Section 4; this is the chain rule
 * through  a = M1 x + b1,  h = GELU(a),  y = M2 h + b2):
 *   db2 = sum_t dy[t]
 *   (dh, dL2, dR2) = adjoints of  y = M2 h  (oracle_bwd with input h)
 *   da = dh * GELU'(a),   GELU'(a) = (1 + erf(a/sqrt 2))/2 + a exp(-a^2/2)/sqrt(2 pi)
 *   db1 = sum_t da[t]
 *   (dx, dL1, dR1) = adjoints of  a = M1 x  (oracle_bwd with output gradient da)
 * All outputs are overwritten.  Any output may be NULL. */
int oracle_mlp_bwd(const double *x, const double *dy, const double *L1, const double *R1,
                   const double *b1, const double *L2, const double *R2, double *dx,
                   double *dL1, double *dR1, double *db1, double *dL2, double *dR2, double *db2,
                   long T, int m)
{
    const size_t n = (size_t)m * m;
    double *a = (double *)malloc((size_t)T * n * sizeof(double));
    double *h = (double *)malloc((size_t)T * n * sizeof(double));
    double *dh = (double *)malloc((size_t)T * n * sizeof(double));
    int fail = !a || !h || !dh;
    if (!fail) fail = oracle_fwd(x, L1, R1, a, NULL, T, m);
    if (!fail) {
#pragma omp parallel for schedule(static)
        for (long t = 0; t < T; ++t)
            for (size_t q = 0; q < n; ++q) {
                const double v = a[(size_t)t * n + q] + b1[q];
                a[(size_t)t * n + q] = v;
                h[(size_t)t * n + q] = 0.5 * v * (1.0 + erf(v / sqrt(2.0)));
            }
        fail = oracle_bwd(h, dy, L2, R2, dh, dL2, dR2, T, m);
    }
    if (!fail) {
        const double inv_sqrt_2pi = 1.0 / sqrt(2.0 * acos(-1.0));
#pragma omp parallel for schedule(static)
        for (long t = 0; t < T; ++t)
            for (size_t q = 0; q < n; ++q) {
                const double v = a[(size_t)t * n + q];
                const double g = 0.5 * (1.0 + erf(v / sqrt(2.0))) + v * exp(-0.5 * v * v) * inv_sqrt_2pi;
                dh[(size_t)t * n + q] *= g;                 /* now da */
            }
        if (db1) {
#pragma omp parallel for schedule(static)
            for (size_t q = 0; q < n; ++q) {
                double acc = 0.0;
                for (long t = 0; t < T; ++t) acc += dh[(size_t)t * n + q];
                db1[q] = acc;
            }
        }
        if (db2) {
#pragma omp parallel for schedule(static)
            for (size_t q = 0; q < n; ++q) {
                double acc = 0.0;
                for (long t = 0; t < T; ++t) acc += dy[(size_t)t * n + q];
                db2[q] = acc;
            }
        }
        fail = oracle_bwd(x, dh, L1, R1, dx, dL1, dR1, T, m);
    }
    free(a);
    free(h);
    free(dh);
    return fail;
}

/* General (rectangular) Monarch multiply, Appendix "General Monarch Matrix
 * Parametrization": M = L R with
 *   R = diag(R_0 .. R_{q-1}),  R_k of size b x b1      (n1 = q b1 inputs, n2 = q b)
 *   L of size n3 x n2 (n3 = r b), a grid of r x q blocks S_{l,k}, each a
 *   b x b diagonal matrix (the case b2 = b3 = b of the rectangular definition,
 *   the one its block-diagonalisation theorem covers).
 * With i = (i1, i0)_b the theorem's blocks are  R'_{i0}[i1][j1] = S_{i1,j1}[i0][i0];
 * they are stored as  Lp[j][l][k] = S_{l,k}[j][j]  (b blocks of r x q).  Then
 *   u[k*b + j] = sum_i R[k][j][i] x[k*b1 + i]         (block-diagonal product)
 *   y[l*b + j] = sum_k Lp[j][l][k] u[k*b + j]         (row l*b+j of L has its
 *                                                      nonzeros in columns k*b+j)
 * q = b1 = b = r = m gives Definition 3.1's square case. */
int oracle_rect_fwd(const double *x, const double *Lp, const double *R, double *y,
                    long T, int q, int b1, int b, int r)
{
    const size_t n1 = (size_t)q * b1, n2 = (size_t)q * b, n3 = (size_t)r * b;
    int fail = 0;
#pragma omp parallel
    {
        double *u = (double *)malloc((n2 ? n2 : 1) * sizeof(double));
        if (!u) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(static)
            for (long t = 0; t < T; ++t) {
                const double *xt = x + (size_t)t * n1;
                double *yt = y + (size_t)t * n3;
                for (int k = 0; k < q; ++k)
                    for (int j = 0; j < b; ++j) {
                        double acc = 0.0;
                        for (int i = 0; i < b1; ++i)
                            acc += R[((size_t)k * b + j) * b1 + i] * xt[(size_t)k * b1 + i];
                        u[(size_t)k * b + j] = acc;
                    }
                for (int l = 0; l < r; ++l)
                    for (int j = 0; j < b; ++j) {
                        double acc = 0.0;
                        for (int k = 0; k < q; ++k)
                            acc += Lp[((size_t)j * r + l) * q + k] * u[(size_t)k * b + j];
                        yt[(size_t)l * b + j] = acc;
                    }
            }
        }
        free(u);
    }
    return fail;
}

/* Gradients of  f = <dy, L R x>  for the general (rectangular) class above - the
 * adjoints of its two steps (the paper trains these layers by automatic
 * differentiation, Section 4):
 *   du[k*b + j]   = sum_l Lp[j][l][k] dy[l*b + j]
 *   dx[k*b1 + i]  = sum_j R[k][j][i]  du[k*b + j]
 *   dLp[j][l][k]  = sum_t dy[t][l*b + j] u[t][k*b + j]
 *   dR[k][j][i]   = sum_t du[t][k*b + j] x[t][k*b1 + i]
 * Any of dx, dLp, dR may be NULL; dLp and dR are overwritten. */
int oracle_rect_bwd(const double *x, const double *dy, const double *Lp, const double *R,
                    double *dx, double *dLp, double *dR, long T, int q, int b1, int b, int r)
{
    const size_t n1 = (size_t)q * b1, n2 = (size_t)q * b, n3 = (size_t)r * b;
    double *u = (double *)malloc(((size_t)T * n2 + 1) * sizeof(double));
    double *du = (double *)malloc(((size_t)T * n2 + 1) * sizeof(double));
    if (!u || !du) {
        free(u);
        free(du);
        return 1;
    }
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        const double *xt = x + (size_t)t * n1, *dyt = dy + (size_t)t * n3;
        double *ut = u + (size_t)t * n2, *dut = du + (size_t)t * n2;
        for (int k = 0; k < q; ++k)
            for (int j = 0; j < b; ++j) {
                double acc = 0.0, dacc = 0.0;
                for (int i = 0; i < b1; ++i)
                    acc += R[((size_t)k * b + j) * b1 + i] * xt[(size_t)k * b1 + i];
                for (int l = 0; l < r; ++l)
                    dacc += Lp[((size_t)j * r + l) * q + k] * dyt[(size_t)l * b + j];
                ut[(size_t)k * b + j] = acc;
                dut[(size_t)k * b + j] = dacc;
            }
        if (dx) {
            double *dxt = dx + (size_t)t * n1;
            for (int k = 0; k < q; ++k)
                for (int i = 0; i < b1; ++i) {
                    double acc = 0.0;
                    for (int j = 0; j < b; ++j)
                        acc += R[((size_t)k * b + j) * b1 + i] * dut[(size_t)k * b + j];
                    dxt[(size_t)k * b1 + i] = acc;
                }
        }
    }
    if (dLp) {
#pragma omp parallel for schedule(static)
        for (int j = 0; j < b; ++j)
            for (int l = 0; l < r; ++l)
                for (int k = 0; k < q; ++k) {
                    double acc = 0.0;
                    for (long t = 0; t < T; ++t)
                        acc += dy[(size_t)t * n3 + (size_t)l * b + j] * u[(size_t)t * n2 + (size_t)k * b + j];
                    dLp[((size_t)j * r + l) * q + k] = acc;
                }
    }
    if (dR) {
#pragma omp parallel for schedule(static)
        for (int k = 0; k < q; ++k)
            for (int j = 0; j < b; ++j)
                for (int i = 0; i < b1; ++i) {
                    double acc = 0.0;
                    for (long t = 0; t < T; ++t)
                        acc += du[(size_t)t * n2 + (size_t)k * b + j] * x[(size_t)t * n1 + (size_t)k * b1 + i];
                    dR[((size_t)k * b + j) * b1 + i] = acc;
                }
    }
    free(u);
    free(du);
    return 0;
}
