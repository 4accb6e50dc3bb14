// Generic Riccati-backward + rollout kernel: one CTA per instance, every matrix of the
// instance resident in shared memory, fp32 FFMA.  Works for any 1 <= n, m <= 64 and is the
// fallback for shapes without a specialised kernel.
//
// Per step t = H-1..0 (Prop. 3.1; Alg. 1 backward loop):
//   V = P B, T = P A, S = R + B'V, Y = B'T, S = L L', K_t = -S^{-1} Y, P_t = Q + A'T + Y'K_t
// then the forward rollout of Alg. 1: u_t = K_t x_t, x_{t+1} = A x_t + B u_t.
#pragma once

#include "common.cuh"

namespace ttc {

// C[M x N] = Cinit + op(A) * B with A read transposed when TA (A stored K x M).
// 4x4 register tiles, ragged edges guarded.  All operands in shared memory.  Cinit may alias C.
template <bool TA>
__device__ __forceinline__ void smem_gemm(int M, int N, int K, const float* A, int lda,
                                          const float* B, int ldb, float* C, int ldc,
                                          const float* Cinit, int ldi)
{
    const int tn = (N + 3) >> 2, tm = (M + 3) >> 2;
    for (int tile = threadIdx.x; tile < tm * tn; tile += blockDim.x) {
        const int i0 = (tile / tn) * 4, j0 = (tile % tn) * 4;
        int ii[4], jj[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            ii[r] = min(i0 + r, M - 1);
            jj[r] = min(j0 + r, N - 1);
        }
        float acc[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c)
                acc[r][c] = 0.f;
        for (int k = 0; k < K; ++k) {
            float a[4], b[4];
#pragma unroll
            for (int r = 0; r < 4; ++r)
                a[r] = TA ? A[k * lda + ii[r]] : A[ii[r] * lda + k];
#pragma unroll
            for (int c = 0; c < 4; ++c)
                b[c] = B[k * ldb + jj[c]];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (i0 + r < M && j0 + c < N) {
                    float v = acc[r][c];
                    if (Cinit)
                        v += Cinit[(i0 + r) * ldi + j0 + c];
                    C[(i0 + r) * ldc + j0 + c] = v;
                }
    }
}

// In-place lower Cholesky of S (m x m, shared memory).  `col` is an m-float scratch.
// Returns 0 or (1-based) index of the first non-positive pivot; the value is uniform
// across the CTA.  Ends with a __syncthreads().
__device__ __forceinline__ int smem_cholesky(int m, float* S, float* col)
{
    for (int j = 0; j < m; ++j) {
        __syncthreads();
        const float d = S[j * m + j];
        if (!(d > 0.f))
            return j + 1;
        const float l = sqrtf(d);
        const float inv = 1.f / l;
        for (int i = j + 1 + threadIdx.x; i < m; i += blockDim.x) {
            const float v = S[i * m + j] * inv;
            S[i * m + j] = v;
            col[i] = v;
        }
        __syncthreads();
        if (threadIdx.x == 0)
            S[j * m + j] = l;
        const int rem = m - j - 1;
        for (int e = threadIdx.x; e < rem * rem; e += blockDim.x) {
            const int i = j + 1 + e / rem, k = j + 1 + e % rem;
            if (k <= i)
                S[i * m + k] = fmaf(-col[i], col[k], S[i * m + k]);
        }
    }
    __syncthreads();
    return 0;
}

// X (m x n, shared) <- -(L L')^{-1} X, one thread per column.
__device__ __forceinline__ void smem_chol_solve_neg(int m, int n, const float* L, float* X)
{
    for (int c = threadIdx.x; c < n; c += blockDim.x) {
        for (int i = 0; i < m; ++i) {
            float v = X[i * n + c];
            for (int k = 0; k < i; ++k)
                v = fmaf(-L[i * m + k], X[k * n + c], v);
            X[i * n + c] = v / L[i * m + i];
        }
        for (int i = m - 1; i >= 0; --i) {
            float v = X[i * n + c];
            for (int k = i + 1; k < m; ++k)
                v = fmaf(-L[k * m + i], X[k * n + c], v);
            X[i * n + c] = v / L[i * m + i];
        }
        for (int i = 0; i < m; ++i)
            X[i * n + c] = -X[i * n + c];
    }
}

// y[rows] = M[rows x cols] * v (+ M2 * v2); M in shared or global, one warp per row group.
__device__ __forceinline__ float warp_dot(const float* row, const float* v, int cols)
{
    float s = 0.f;
    for (int j = threadIdx.x & 31; j < cols; j += 32)
        s = fmaf(row[j], v[j], s);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        s += __shfl_xor_sync(0xffffffffu, s, o);
    return s;
}

// Forward rollout of Alg. 1 for one instance by one CTA.  Kt_src: gains [H][m][n] in global
// memory (or, when only u_0 is wanted, the K_0 left in shared memory: pass Ksm and H_roll = 1).
__device__ __forceinline__ void cta_rollout(const SolveParams& p, long long inst, float* sA,
                                            float* sB, const float* Kglob, const float* Ksm,
                                            float* sx, float* sxn, float* su, int steps,
                                            const float* kglob = nullptr, const float* ksm = nullptr)
{
    const int n = p.n, m = p.m, H = p.H;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    float* xo = p.x ? p.x + inst * (long long)(H + 1) * n : nullptr;
    float* uo = p.u ? p.u + inst * (long long)(p.first_only ? m : H * m) : nullptr;
    if (xo)
        for (int e = threadIdx.x; e < n; e += blockDim.x)
            xo[e] = sx[e];
    for (int t = 0; t < steps; ++t) {
        const float* Kt = Ksm ? Ksm : Kglob + (long long)t * m * n;
        if (p.A.st || p.B.st) {                      // time-varying dynamics: A_t, B_t of this step
            if (p.A.st)
                load_to_smem(sA, p.A, operand_offset(p.A, inst, p.b1, p.b2) + t * p.A.st, n * n);
            if (p.B.st)
                load_to_smem(sB, p.B, operand_offset(p.B, inst, p.b1, p.b2) + t * p.B.st, n * m);
            __syncthreads();
        }
        const float* kt = ksm ? ksm : (kglob ? kglob + (long long)t * m : nullptr);     // u_t = K_t x_t + k_t
        for (int i = warp; i < m; i += nw) {
            const float s = warp_dot(Kt + i * n, sx, n);
            if (lane == 0)
                su[i] = kt ? s + kt[i] : s;
        }
        __syncthreads();
        for (int i = warp; i < n; i += nw) {
            const float s = warp_dot(sA + i * n, sx, n) + warp_dot(sB + i * m, su, m);
            if (lane == 0)
                sxn[i] = s;
        }
        __syncthreads();
        if (uo && (!p.first_only || t == 0))
            for (int e = threadIdx.x; e < m; e += blockDim.x)
                uo[(p.first_only ? 0 : t * m) + e] = su[e];
        if (xo)
            for (int e = threadIdx.x; e < n; e += blockDim.x)
                xo[(long long)(t + 1) * n + e] = sxn[e];
        for (int e = threadIdx.x; e < n; e += blockDim.x)
            sx[e] = sxn[e];
        __syncthreads();
    }
}

// Fill every requested output of one instance with quiet NaN and record `code`.
__device__ __forceinline__ void cta_fail_instance(const SolveParams& p, long long inst, int code)
{
    const int n = p.n, m = p.m, H = p.H;
    const float qn = quiet_nan();
    if (p.K)
        for (long long e = threadIdx.x; e < (long long)H * m * n; e += blockDim.x)
            p.K[inst * (long long)H * m * n + e] = qn;
    if (p.P) {
        const long long cnt = (long long)(p.first_only ? 1 : H + 1) * n * n;
        for (long long e = threadIdx.x; e < cnt; e += blockDim.x)
            p.P[inst * cnt + e] = qn;
    }
    if (p.x)
        for (long long e = threadIdx.x; e < (long long)(H + 1) * n; e += blockDim.x)
            p.x[inst * (long long)(H + 1) * n + e] = qn;
    if (p.u) {
        const long long cnt = p.first_only ? m : (long long)H * m;
        for (long long e = threadIdx.x; e < cnt; e += blockDim.x)
            p.u[inst * cnt + e] = qn;
    }
    if (p.pvec) {
        const long long cnt = (long long)(p.first_only ? 1 : H + 1) * n;
        for (long long e = threadIdx.x; e < cnt; e += blockDim.x)
            p.pvec[inst * cnt + e] = qn;
    }
    if (p.kff && p.r.ptr)
        for (long long e = threadIdx.x; e < (long long)H * m; e += blockDim.x)
            p.kff[inst * (long long)H * m + e] = qn;
    if (p.info && threadIdx.x == 0)
        p.info[inst] = code;
}

inline size_t riccati_cta_smem_bytes(int n, int m)
{
    // A, Q, P, T: n*n ; B, V, Y, K: n*m ; R, S: m*m ; x, xn, p: n ; u, col, g: m
    return sizeof(float) * (size_t)(4 * n * n + 4 * n * m + 2 * m * m + 3 * n + 3 * m);
}

__global__ void __launch_bounds__(256) riccati_cta_kernel(SolveParams p)
{
    extern __shared__ __align__(16) float sm[];
    const int n = p.n, m = p.m, H = p.H;
    float* sA = sm;
    float* sQ = sA + n * n;
    float* sP = sQ + n * n;
    float* sT = sP + n * n;
    float* sB = sT + n * n;
    float* sV = sB + n * m;
    float* sY = sV + n * m;
    float* sK = sY + n * m;
    float* sR = sK + n * m;
    float* sS = sR + m * m;
    float* sx = sS + m * m;
    float* sxn = sx + n;
    float* su = sxn + n;
    float* scol = su + m;
    float* sp = scol + m;      // p_{t+1} of the affine recursion (Prop. A.1)
    float* sg = sp + n;        // B'p + r, then k_t

    for (long long widx = blockIdx.x; widx < p.b0 * p.b1 * p.tcount; widx += gridDim.x) {
        const long long inst = window_instance(p, widx);
        __syncthreads();
        for (int e = threadIdx.x; e < n; e += blockDim.x)
            sp[e] = 0.f;                                          // p_H = 0
        load_to_smem(sA, p.A, operand_offset(p.A, inst, p.b1, p.b2), n * n);
        load_to_smem(sB, p.B, operand_offset(p.B, inst, p.b1, p.b2), n * m);
        load_to_smem(sR, p.R, operand_offset(p.R, inst, p.b1, p.b2), m * m);
        {
            const long long oq = operand_offset(p.Q, inst, p.b1, p.b2);
            const long long of = p.Qf.ptr ? operand_offset(p.Qf, inst, p.b1, p.b2) : 0;
            for (int e = threadIdx.x; e < n * n; e += blockDim.x) {
                sQ[e] = load_elem(p.Q, oq + e);
                sP[e] = p.Qf.ptr ? load_elem(p.Qf, of + e) : sQ[e];       // P_H = Q_f
            }
        }
        if (p.x0.ptr)
            load_to_smem(sx, p.x0, operand_offset(p.x0, inst, p.b1, p.b2), n);
        __syncthreads();

        float* Kout = p.K ? p.K + inst * (long long)H * m * n
                          : (p.Kws ? p.Kws + inst * (long long)H * m * n : nullptr);
        float* Pout = p.P ? p.P + inst * (long long)(p.first_only ? 1 : H + 1) * n * n : nullptr;
        if (Pout && !p.first_only)
            for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                Pout[(long long)H * n * n + e] = sP[e];      // P_H
        if (p.pvec && !p.first_only)
            for (int e = threadIdx.x; e < n; e += blockDim.x)
                p.pvec[inst * (long long)(H + 1) * n + (long long)H * n + e] = 0.f;

        int fail = 0;
        for (int t = H - 1; t >= 0; --t) {
            if (p.A.st || p.B.st || p.Q.st || p.R.st) {                      // time-varying operands of step t
                if (p.A.st) load_to_smem(sA, p.A, operand_offset(p.A, inst, p.b1, p.b2) + t * p.A.st, n * n);
                if (p.B.st) load_to_smem(sB, p.B, operand_offset(p.B, inst, p.b1, p.b2) + t * p.B.st, n * m);
                if (p.R.st) load_to_smem(sR, p.R, operand_offset(p.R, inst, p.b1, p.b2) + t * p.R.st, m * m);
                if (p.Q.st) load_to_smem(sQ, p.Q, operand_offset(p.Q, inst, p.b1, p.b2) + t * p.Q.st, n * n);
                __syncthreads();
            }
            smem_gemm<false>(n, m, n, sP, n, sB, m, sV, m, nullptr, 0);      // V = P B
            smem_gemm<false>(n, n, n, sP, n, sA, n, sT, n, nullptr, 0);      // T = P A
            __syncthreads();
            smem_gemm<true>(m, m, n, sB, m, sV, m, sS, m, sR, m);            // S = R + B'V
            smem_gemm<true>(m, n, n, sB, m, sT, n, sY, n, nullptr, 0);       // Y = B'T
            __syncthreads();
            const int bad = smem_cholesky(m, sS, scol);
            if (bad) {
                fail = t * m + bad;
                break;
            }
            for (int e = threadIdx.x; e < m * n; e += blockDim.x)
                sK[e] = sY[e];
            __syncthreads();
            smem_chol_solve_neg(m, n, sS, sK);                               // K = -S^{-1} Y
            __syncthreads();
            smem_gemm<true>(n, n, n, sA, n, sT, n, sP, n, sQ, n);            // P = Q + A'T
            __syncthreads();
            smem_gemm<true>(n, n, m, sY, n, sK, n, sP, n, sP, n);            // P += Y'K
            __syncthreads();
            for (int e = threadIdx.x; e < n * n; e += blockDim.x) {          // symmetrise
                const int i = e / n, j = e % n;
                if (i < j) {
                    const float s = 0.5f * (sP[i * n + j] + sP[j * n + i]);
                    sP[i * n + j] = s;
                    sP[j * n + i] = s;
                }
            }
            __syncthreads();
            if (Kout)
                for (int e = threadIdx.x; e < m * n; e += blockDim.x)
                    Kout[(long long)t * m * n + e] = sK[e];
            if (Pout && (!p.first_only || t == 0))
                for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                    Pout[(long long)(p.first_only ? 0 : t) * n * n + e] = sP[e];
            if (p.r.ptr) {
                // linear control cost (Prop. A.1): k_t = -S^{-1}(B'p_{t+1} + r_t), p_t = A'p_{t+1} + Y'k_t
                const long long orv = operand_offset(p.r, inst, p.b1, p.b2) + t * p.r.st;
                for (int e = threadIdx.x; e < m; e += blockDim.x) {
                    float g = t < p.r_count ? load_elem(p.r, orv + e) : 0.f;
                    for (int k = 0; k < n; ++k)
                        g = fmaf(sB[k * m + e], sp[k], g);
                    sg[e] = g;
                }
                __syncthreads();
                smem_chol_solve_neg(m, 1, sS, sg);
                __syncthreads();
                float pn = 0.f;
                const int i = threadIdx.x;
                if (i < n) {
                    for (int k = 0; k < n; ++k)
                        pn = fmaf(sA[k * n + i], sp[k], pn);
                    for (int k = 0; k < m; ++k)
                        pn = fmaf(sY[k * n + i], sg[k], pn);
                }
                __syncthreads();
                if (i < n) {
                    sp[i] = pn;
                    if (p.pvec && (!p.first_only || t == 0))
                        p.pvec[inst * (long long)(p.first_only ? 1 : H + 1) * n + (long long)(p.first_only ? 0 : t) * n + i] = pn;
                }
                if (p.kff)
                    for (int e = threadIdx.x; e < m; e += blockDim.x)
                        p.kff[(inst * (long long)H + t) * m + e] = sg[e];
            }
        }
        if (fail) {
            __syncthreads();
            cta_fail_instance(p, inst, fail);
            continue;
        }
        if (p.info && threadIdx.x == 0)
            p.info[inst] = 0;
        if (p.x || p.u) {
            __syncthreads();   // K_t written by this CTA are visible to it after the barrier
            const bool only_u0 = p.first_only && !p.x;
            const float* kglob = (p.r.ptr && p.kff) ? p.kff + inst * (long long)H * m : nullptr;
            cta_rollout(p, inst, sA, sB, Kout, only_u0 ? sK : nullptr, sx, sxn, su, only_u0 ? 1 : H, kglob,
                        (only_u0 && p.r.ptr) ? sg : nullptr);
        }
    }
}

} // namespace ttc
