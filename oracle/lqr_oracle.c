/*
 * lqr_oracle.c -- float64 CPU oracle for the batched finite-horizon LQR solve.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code, header, table or helper
 * with the CUDA path and must never be called from it.  Only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may use it.
 *
 * What it computes (library indexing: x_{t+1} = A x_t + B u_t, t = 0..H-1,
 * cost sum_t (x_t'Q x_t + u_t'R u_t) + x_H'Q x_H):
 *
 *   P_H = Q                                             (Prop. 3.1: P_T = Q_T)
 *   for t = H-1 .. 0                                    (Alg. 1, backward loop)
 *     S   = R + B' P_{t+1} B
 *     Y   = B' P_{t+1} A
 *     K_t = -S^{-1} Y                                   (Eq. 4 of Prop. 3.1)
 *     P_t = Q + A' P_{t+1} A + Y' K_t                   (Eq. 5, the Riccati step)
 *     P_t = (P_t + P_t')/2
 *   x_0 given; for t = 0 .. H-1                         (Alg. 1, forward rollout)
 *     u_t = K_t x_t ;  x_{t+1} = A x_t + B u_t
 *
 * Relation to the paper's indexing (h_t = A h_{t-1} + B u_t, t = 1..T, Q_0 = 0):
 * x_t = h_t, u_t = u_{t+1}(paper), K_t = K_{t+1}(paper), P_t = P_t(paper) for
 * t >= 1 and P_0 = P_0(paper) + Q.  S^{-1} is applied through a Cholesky
 * factorisation (S is positive definite when R is and P is semi-definite).
 *
 * Time-varying problems (Definition A.1 with A_t, B_t, Q_t, R_t and a terminal weight Q_f,
 * Prop. A.1 / Alg. 1 with time indices kept): lqr_oracle_solve_tv takes, per operand, the element
 * stride between consecutive time indices (0 = the same matrix at every t):
 *   P_H = Q_f ;  S = R_t + B_t' P_{t+1} B_t ;  Y = B_t' P_{t+1} A_t ;  K_t = -S^{-1} Y ;
 *   P_t = Q_t + A_t' P_{t+1} A_t + Y' K_t ;  u_t = K_t x_t ;  x_{t+1} = A_t x_t + B_t u_t,
 * with cost sum_{t<H} (x_t'Q_t x_t + u_t'R_t u_t) + x_H'Q_f x_H.  The paper's h_t = A_t h_{t-1} + B_t u_t
 * (t = 1..T) maps to x_t = h_t, A_t(here) = A_{t+1}(paper), likewise B and R, Q_t(here) = Q_t(paper),
 * Q_f = Q_T.  The time-invariant entry points are this function with all strides 0 and Q_f = Q.
 *
 * All matrices are row-major and contiguous.  Parity status: pinned (brute-force
 * KKT solve, closed forms, invariants, DARE limit, symplectic cross-identity --
 * see tests/test_oracle_*.py; the time-varying function by a brute-force KKT solve with
 * time-varying blocks, tail consistency and the cost identity -- tests/test_oracle_tv_pins.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* C[M x N] = A'[M x K] * B[K x N] where A is stored K x M (so C = A^T B). */
static void mm_tn(int M, int N, int K, const double *A, const double *B, double *C)
{
    for (int i = 0; i < M; ++i)
        for (int j = 0; j < N; ++j)
            C[i * N + j] = 0.0;
    for (int k = 0; k < K; ++k)
        for (int i = 0; i < M; ++i) {
            double a = A[k * M + i];
            for (int j = 0; j < N; ++j)
                C[i * N + j] += a * B[k * N + j];
        }
}

/* C[M x N] = A[M x K] * B[K x N]. */
static void mm_nn(int M, int N, int K, const double *A, const double *B, double *C)
{
    for (int i = 0; i < M; ++i) {
        for (int j = 0; j < N; ++j)
            C[i * N + j] = 0.0;
        for (int k = 0; k < K; ++k) {
            double a = A[i * K + k];
            for (int j = 0; j < N; ++j)
                C[i * N + j] += a * B[k * N + j];
        }
    }
}

/* In-place lower Cholesky of the m x m matrix S (row-major); returns 0 or the
 * 1-based index of the first non-positive pivot. */
static int chol_lower(int m, double *S)
{
    for (int j = 0; j < m; ++j) {
        double d = S[j * m + j];
        for (int k = 0; k < j; ++k)
            d -= S[j * m + k] * S[j * m + k];
        if (!(d > 0.0))
            return j + 1;
        d = sqrt(d);
        S[j * m + j] = d;
        for (int i = j + 1; i < m; ++i) {
            double v = S[i * m + j];
            for (int k = 0; k < j; ++k)
                v -= S[i * m + k] * S[j * m + k];
            S[i * m + j] = v / d;
        }
    }
    return 0;
}

/* Solve (L L') X = Y for X, Y is m x n (overwritten by X). */
static void chol_solve(int m, int n, const double *L, double *Y)
{
    for (int c = 0; c < n; ++c) {
        for (int i = 0; i < m; ++i) {           /* L z = y */
            double v = Y[i * n + c];
            for (int k = 0; k < i; ++k)
                v -= L[i * m + k] * Y[k * n + c];
            Y[i * n + c] = v / L[i * m + i];
        }
        for (int i = m - 1; i >= 0; --i) {      /* L' x = z */
            double v = Y[i * n + c];
            for (int k = i + 1; k < m; ++k)
                v -= L[k * m + i] * Y[k * n + c];
            Y[i * n + c] = v / L[i * m + i];
        }
    }
}

/*
 * One instance.  Outputs (any may be NULL): K [H][m][n], P [H+1][n][n] (or
 * [n][n] = P_0 when first_only), x [H+1][n], u [H][m] (or [m] = u_0 when
 * first_only).  Returns 0, or t*m + j + 1 when pivot j (0-based) of
 * S = R + B'P_{t+1}B at time index t was not positive; outputs are then
 * unspecified.  Returns -1 on bad sizes / allocation failure.
 */
int lqr_oracle_solve_tv(int n, int m, int H, const double *A0, int64_t sA, const double *B0, int64_t sB,
                        const double *Q0, int64_t sQ, const double *R0, int64_t sR, const double *Qf,
                        const double *x0, double *K, double *P, double *x, double *u, int first_only)
{
    if (n < 1 || m < 1 || H < 1)
        return -1;
    size_t nn = (size_t)n * n, nm = (size_t)n * m, mm = (size_t)m * m;
    double *Pall = (double *)malloc(sizeof(double) * nn * (size_t)(H + 1));
    double *Kall = (double *)malloc(sizeof(double) * nm * (size_t)H);
    double *W = (double *)malloc(sizeof(double) * (3 * nn + 2 * nm + mm + 2 * (size_t)n + m));
    if (!Pall || !Kall || !W) {
        free(Pall); free(Kall); free(W);
        return -1;
    }
    double *PA = W;            /* n x n : P_{t+1} A         */
    double *AtPA = PA + nn;    /* n x n : A' P_{t+1} A      */
    double *YtK = AtPA + nn;   /* n x n : Y' K_t            */
    double *PB = YtK + nn;     /* n x m : P_{t+1} B         */
    double *Y = PB + nm;       /* m x n : B' P_{t+1} A      */
    double *S = Y + nm;        /* m x m : R + B' P_{t+1} B  */
    double *xt = S + mm, *xn = xt + n, *ut = xn + n;
    int info = 0;

    memcpy(Pall + nn * (size_t)H, Qf, sizeof(double) * nn);         /* P_H = Q_f */
    for (int t = H - 1; t >= 0 && info == 0; --t) {
        const double *Pn = Pall + nn * (size_t)(t + 1);
        double *Pt = Pall + nn * (size_t)t;
        double *Kt = Kall + nm * (size_t)t;
        const double *A = A0 + sA * t, *B = B0 + sB * t, *Q = Q0 + sQ * t, *R = R0 + sR * t;
        mm_nn(n, m, n, Pn, B, PB);
        mm_tn(m, m, n, B, PB, S);                                   /* B'(P B)  */
        for (size_t i = 0; i < mm; ++i)
            S[i] += R[i];
        mm_nn(n, n, n, Pn, A, PA);
        mm_tn(m, n, n, B, PA, Y);                                   /* B'(P A)  */
        int bad = chol_lower(m, S);
        if (bad) {
            info = t * m + bad;
            break;
        }
        memcpy(Kt, Y, sizeof(double) * nm);
        chol_solve(m, n, S, Kt);
        for (size_t i = 0; i < nm; ++i)
            Kt[i] = -Kt[i];                                         /* K_t = -S^{-1} Y */
        mm_tn(n, n, n, A, PA, AtPA);
        mm_tn(n, n, m, Y, Kt, YtK);
        for (int i = 0; i < n; ++i)
            for (int j = 0; j < n; ++j)
                Pt[i * n + j] = Q[i * n + j] + AtPA[i * n + j] + YtK[i * n + j];
        for (int i = 0; i < n; ++i)
            for (int j = i + 1; j < n; ++j) {
                double s = 0.5 * (Pt[i * n + j] + Pt[j * n + i]);
                Pt[i * n + j] = s;
                Pt[j * n + i] = s;
            }
    }

    if (info == 0) {
        if (K)
            memcpy(K, Kall, sizeof(double) * nm * (size_t)H);
        if (P)
            memcpy(P, Pall, sizeof(double) * nn * (size_t)(first_only ? 1 : H + 1));
        memcpy(xt, x0, sizeof(double) * (size_t)n);
        if (x)
            memcpy(x, xt, sizeof(double) * (size_t)n);
        for (int t = 0; t < H; ++t) {
            const double *Kt = Kall + nm * (size_t)t;
            const double *A = A0 + sA * t, *B = B0 + sB * t;
            for (int i = 0; i < m; ++i) {
                double s = 0.0;
                for (int j = 0; j < n; ++j)
                    s += Kt[i * n + j] * xt[j];
                ut[i] = s;
            }
            for (int i = 0; i < n; ++i) {
                double s = 0.0;
                for (int j = 0; j < n; ++j)
                    s += A[i * n + j] * xt[j];
                for (int j = 0; j < m; ++j)
                    s += B[i * m + j] * ut[j];
                xn[i] = s;
            }
            if (u && (!first_only || t == 0))
                memcpy(u + (first_only ? 0 : (size_t)t * m), ut, sizeof(double) * (size_t)m);
            if (x)
                memcpy(x + (size_t)(t + 1) * n, xn, sizeof(double) * (size_t)n);
            memcpy(xt, xn, sizeof(double) * (size_t)n);
            if (first_only && !x)
                break;
        }
    }
    free(Pall); free(Kall); free(W);
    return info;
}

/* Time-invariant problem: every stride 0, terminal weight Q (Prop. 3.1 with P_T = Q). */
int lqr_oracle_solve(int n, int m, int H, const double *A, const double *B, const double *Q,
                     const double *R, const double *x0, double *K, double *P, double *x,
                     double *u, int first_only)
{
    return lqr_oracle_solve_tv(n, m, H, A, 0, B, 0, Q, 0, R, 0, Q, x0, K, P, x, u, first_only);
}

/*
 * N independent instances.  off*[i] is the element offset of instance i's
 * operand inside the corresponding base array (this is how operands shared by a
 * head are expressed: equal offsets).  Outputs are dense per instance.
 * Instances are distributed over `nthreads` OpenMP threads.  Returns the number
 * of threads actually used.
 */
int lqr_oracle_solve_batch_tv(int64_t N, int n, int m, int H,
                              const double *A, const int64_t *offA, int64_t sA,
                              const double *B, const int64_t *offB, int64_t sB,
                              const double *Q, const int64_t *offQ, int64_t sQ,
                              const double *R, const int64_t *offR, int64_t sR,
                              const double *Qf, const int64_t *offQf,
                              const double *x0, const int64_t *offx,
                              double *K, double *P, double *x, double *u, int32_t *info,
                              int first_only, int nthreads)
{
    size_t nn = (size_t)n * n, nm = (size_t)n * m;
    size_t sP = first_only ? nn : nn * (size_t)(H + 1);
    size_t su = first_only ? (size_t)m : (size_t)m * H;
    int used = 1;
#ifdef _OPENMP
    if (nthreads < 1)
        nthreads = omp_get_max_threads();
#pragma omp parallel num_threads(nthreads)
    {
#pragma omp single
        used = omp_get_num_threads();
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < N; ++i) {
            int r = lqr_oracle_solve_tv(n, m, H, A + offA[i], sA, B + offB[i], sB, Q + offQ[i], sQ, R + offR[i], sR,
                                     Qf + offQf[i], x0 + offx[i], K ? K + (size_t)i * nm * H : NULL,
                                     P ? P + (size_t)i * sP : NULL,
                                     x ? x + (size_t)i * n * (H + 1) : NULL,
                                     u ? u + (size_t)i * su : NULL, first_only);
            if (info)
                info[i] = r;
        }
    }
#else
    (void)nthreads;
    for (int64_t i = 0; i < N; ++i) {
        int r = lqr_oracle_solve_tv(n, m, H, A + offA[i], sA, B + offB[i], sB, Q + offQ[i], sQ, R + offR[i], sR,
                                 Qf + offQf[i], x0 + offx[i], K ? K + (size_t)i * nm * H : NULL,
                                 P ? P + (size_t)i * sP : NULL,
                                 x ? x + (size_t)i * n * (H + 1) : NULL,
                                 u ? u + (size_t)i * su : NULL, first_only);
        if (info)
            info[i] = r;
    }
#endif
    return used;
}

/* Time-invariant batch: strides 0, Q_f = Q. */
int lqr_oracle_solve_batch(int64_t N, int n, int m, int H,
                           const double *A, const int64_t *offA,
                           const double *B, const int64_t *offB,
                           const double *Q, const int64_t *offQ,
                           const double *R, const int64_t *offR,
                           const double *x0, const int64_t *offx,
                           double *K, double *P, double *x, double *u, int32_t *info,
                           int first_only, int nthreads)
{
    return lqr_oracle_solve_batch_tv(N, n, m, H, A, offA, 0, B, offB, 0, Q, offQ, 0, R, offR, 0, Q, offQ,
                                     x0, offx, K, P, x, u, info, first_only, nthreads);
}

/*
 * Affine control cost (Definition A.1 with r_t; Prop. A.1): stage cost
 *     1/2 (x_t'Q_t x_t + u_t'R_t u_t) + r_t'u_t,  terminal cost 1/2 x_H'Q_f x_H
 * (with the linear term the factor 1/2 matters; P_t and K_t are those of lqr_oracle_solve_tv).
 * Value function V_t(x) = 1/2 x'P_t x + p_t'x + c_t, p_H = 0, and for t = H-1..0 with
 * S = R_t + B_t'P_{t+1}B_t, Y = B_t'P_{t+1}A_t:
 *     K_t = -S^{-1} Y,                 k_t = -S^{-1} (B_t'p_{t+1} + r_t),
 *     P_t = Q_t + A_t'P_{t+1}A_t + Y'K_t,   p_t = A_t'p_{t+1} + Y'k_t,
 * then u_t = K_t x_t + k_t, x_{t+1} = A_t x_t + B_t u_t.
 * r0: [H][m] with element stride sr between time indices (0 = the same vector at every t).
 * Outputs (any may be NULL): K [H][m][n], kff [H][m], P [H+1][n][n], pvec [H+1][n], x [H+1][n], u [H][m].
 * Returns as lqr_oracle_solve_tv.
 */
int lqr_oracle_solve_affine(int n, int m, int H, const double *A0, int64_t sA, const double *B0, int64_t sB,
                            const double *Q0, int64_t sQ, const double *R0, int64_t sR, const double *r0, int64_t sr,
                            const double *Qf, const double *x0, double *K, double *kff, double *P, double *pvec,
                            double *x, double *u)
{
    if (n < 1 || m < 1 || H < 1)
        return -1;
    size_t nn = (size_t)n * n, nm = (size_t)n * m, mm = (size_t)m * m;
    double *Pall = (double *)malloc(sizeof(double) * nn * (size_t)(H + 1));
    double *pall = (double *)calloc((size_t)n * (size_t)(H + 1), sizeof(double));
    double *Kall = (double *)malloc(sizeof(double) * nm * (size_t)H);
    double *kall = (double *)malloc(sizeof(double) * (size_t)m * (size_t)H);
    double *W = (double *)malloc(sizeof(double) * (3 * nn + 2 * nm + mm + 2 * (size_t)n + 2 * (size_t)m));
    if (!Pall || !pall || !Kall || !kall || !W) {
        free(Pall); free(pall); free(Kall); free(kall); free(W);
        return -1;
    }
    double *PA = W, *AtPA = PA + nn, *YtK = AtPA + nn, *PB = YtK + nn, *Y = PB + nm, *S = Y + nm;
    double *xt = S + mm, *xn = xt + n, *ut = xn + n, *g = ut + m;
    int info = 0;

    memcpy(Pall + nn * (size_t)H, Qf, sizeof(double) * nn);         /* P_H = Q_f, p_H = 0 */
    for (int t = H - 1; t >= 0 && info == 0; --t) {
        const double *Pn = Pall + nn * (size_t)(t + 1), *pn = pall + (size_t)n * (size_t)(t + 1);
        double *Pt = Pall + nn * (size_t)t, *pt = pall + (size_t)n * (size_t)t;
        double *Kt = Kall + nm * (size_t)t, *kt = kall + (size_t)m * (size_t)t;
        const double *A = A0 + sA * t, *B = B0 + sB * t, *Q = Q0 + sQ * t, *R = R0 + sR * t, *r = r0 + sr * t;
        mm_nn(n, m, n, Pn, B, PB);
        mm_tn(m, m, n, B, PB, S);
        for (size_t i = 0; i < mm; ++i)
            S[i] += R[i];
        mm_nn(n, n, n, Pn, A, PA);
        mm_tn(m, n, n, B, PA, Y);
        int bad = chol_lower(m, S);
        if (bad) {
            info = t * m + bad;
            break;
        }
        memcpy(Kt, Y, sizeof(double) * nm);
        chol_solve(m, n, S, Kt);
        for (size_t i = 0; i < nm; ++i)
            Kt[i] = -Kt[i];
        for (int i = 0; i < m; ++i) {                               /* g = B'p_{t+1} + r_t */
            double s = r[i];
            for (int k = 0; k < n; ++k)
                s += B[k * m + i] * pn[k];
            g[i] = s;
        }
        memcpy(kt, g, sizeof(double) * (size_t)m);
        chol_solve(m, 1, S, kt);
        for (int i = 0; i < m; ++i)
            kt[i] = -kt[i];                                         /* k_t = -S^{-1} g */
        mm_tn(n, n, n, A, PA, AtPA);
        mm_tn(n, n, m, Y, Kt, YtK);
        for (int i = 0; i < n; ++i)
            for (int j = 0; j < n; ++j)
                Pt[i * n + j] = Q[i * n + j] + AtPA[i * n + j] + YtK[i * n + j];
        for (int i = 0; i < n; ++i)
            for (int j = i + 1; j < n; ++j) {
                double s = 0.5 * (Pt[i * n + j] + Pt[j * n + i]);
                Pt[i * n + j] = s;
                Pt[j * n + i] = s;
            }
        for (int i = 0; i < n; ++i) {                               /* p_t = A'p_{t+1} + Y'k_t */
            double s = 0.0;
            for (int k = 0; k < n; ++k)
                s += A[k * n + i] * pn[k];
            for (int k = 0; k < m; ++k)
                s += Y[k * n + i] * kt[k];
            pt[i] = s;
        }
    }
    if (info == 0) {
        if (K) memcpy(K, Kall, sizeof(double) * nm * (size_t)H);
        if (kff) memcpy(kff, kall, sizeof(double) * (size_t)m * (size_t)H);
        if (P) memcpy(P, Pall, sizeof(double) * nn * (size_t)(H + 1));
        if (pvec) memcpy(pvec, pall, sizeof(double) * (size_t)n * (size_t)(H + 1));
        memcpy(xt, x0, sizeof(double) * (size_t)n);
        if (x) memcpy(x, xt, sizeof(double) * (size_t)n);
        for (int t = 0; t < H; ++t) {
            const double *Kt = Kall + nm * (size_t)t, *kt = kall + (size_t)m * (size_t)t;
            const double *A = A0 + sA * t, *B = B0 + sB * t;
            for (int i = 0; i < m; ++i) {
                double s = kt[i];
                for (int j = 0; j < n; ++j)
                    s += Kt[i * n + j] * xt[j];
                ut[i] = s;
            }
            for (int i = 0; i < n; ++i) {
                double s = 0.0;
                for (int j = 0; j < n; ++j)
                    s += A[i * n + j] * xt[j];
                for (int j = 0; j < m; ++j)
                    s += B[i * m + j] * ut[j];
                xn[i] = s;
            }
            if (u) memcpy(u + (size_t)t * m, ut, sizeof(double) * (size_t)m);
            if (x) memcpy(x + (size_t)(t + 1) * n, xn, sizeof(double) * (size_t)n);
            memcpy(xt, xn, sizeof(double) * (size_t)n);
        }
    }
    free(Pall); free(pall); free(Kall); free(kall); free(W);
    return info;
}
