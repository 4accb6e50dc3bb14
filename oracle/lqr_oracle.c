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
 * All matrices are row-major and contiguous.  Parity status: pinned (brute-force
 * KKT solve, closed forms, invariants, DARE limit, symplectic cross-identity --
 * see tests/test_oracle_*.py).
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
int lqr_oracle_solve(int n, int m, int H, const double *A, const double *B, const double *Q,
                     const double *R, const double *x0, double *K, double *P, double *x,
                     double *u, int first_only)
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

    memcpy(Pall + nn * (size_t)H, Q, sizeof(double) * nn);          /* P_H = Q */
    for (int t = H - 1; t >= 0 && info == 0; --t) {
        const double *Pn = Pall + nn * (size_t)(t + 1);
        double *Pt = Pall + nn * (size_t)t;
        double *Kt = Kall + nm * (size_t)t;
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

/*
 * N independent instances.  off*[i] is the element offset of instance i's
 * operand inside the corresponding base array (this is how operands shared by a
 * head are expressed: equal offsets).  Outputs are dense per instance.
 * Instances are distributed over `nthreads` OpenMP threads.  Returns the number
 * of threads actually used.
 */
int lqr_oracle_solve_batch(int64_t N, int n, int m, int H,
                           const double *A, const int64_t *offA,
                           const double *B, const int64_t *offB,
                           const double *Q, const int64_t *offQ,
                           const double *R, const int64_t *offR,
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
            int r = lqr_oracle_solve(n, m, H, A + offA[i], B + offB[i], Q + offQ[i], R + offR[i],
                                     x0 + offx[i], K ? K + (size_t)i * nm * H : NULL,
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
        int r = lqr_oracle_solve(n, m, H, A + offA[i], B + offB[i], Q + offQ[i], R + offR[i],
                                 x0 + offx[i], K ? K + (size_t)i * nm * H : NULL,
                                 P ? P + (size_t)i * sP : NULL,
                                 x ? x + (size_t)i * n * (H + 1) : NULL,
                                 u ? u + (size_t)i * su : NULL, first_only);
        if (info)
            info[i] = r;
    }
#endif
    return used;
}
