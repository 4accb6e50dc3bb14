// Symplectic-pair scan over the horizon, and the fused gain + rollout kernel.
//
// The transition of [state; co-state] over one step is the symplectic matrix S_t of
// Thm A.2.  It is stored inverse-free as the triple e = (A, C, J) with C = B R^{-1} B' and
// J = Q, for which  M(e) = [[A + C A^{-T} J, -C A^{-T}], [-A^{-T} J, A^{-T}]] = S_t.
// Composing two transitions (e1 first, e2 second; M(e1 o e2) = M(e2) M(e1)) is, in blocks,
//     W = (I + C1 J2)^{-1}
//     A12 = A2 W A1,   C12 = A2 W C1 A2' + C2,   J12 = A1' J2 W A1 + J1
// and the map an element induces on value matrices is
//     apply(e, P) = J + A' (I + P C)^{-1} P A          (one step: the Riccati step).
// Neither needs A^{-1}; I + C J has eigenvalues >= 1 for PSD C, J.
//
// Time-invariant problem => all step elements are equal and the suffix products are powers:
// P_{H-k} = apply(e^k, Q).  Round r holds e^(2^r) and produces P_{H-k} for 2^r <= k < 2^(r+1)
// from P_{H-k+2^r}; then e^(2^(r+1)) = e^(2^r) o e^(2^r).  Depth log2(H) instead of H.
// When only P_0 / u_0 are wanted, P_1 = apply(e^(H-1), Q) follows the binary digits of H-1.
//
// Linear systems are solved by Gauss-Jordan elimination with partial pivoting on the
// augmented matrix in shared memory.
#pragma once

#include "common.cuh"
#include "riccati_cta.cuh"

namespace ttc {

// Gauss-Jordan with partial pivoting on W = [M | RHS] (n rows, n + r columns, row stride ldw).
// On return X[i][c] = W[i][n + c] / W[i][i] solves M X = RHS.  Returns 0 or the 1-based column
// at which no non-zero pivot was found (uniform across the CTA).  Ends with __syncthreads().
__device__ __forceinline__ int smem_gauss_jordan(int n, int r, float* W, int ldw)
{
    const int cols = n + r;
    for (int j = 0; j < n; ++j) {
        __syncthreads();
        if (threadIdx.x < 32) {
            const int lane = threadIdx.x;
            float best = -1.f;
            int bi = j;
            for (int i = j + lane; i < n; i += 32) {
                const float a = fabsf(W[i * ldw + j]);
                if (a > best) {
                    best = a;
                    bi = i;
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ob = __shfl_xor_sync(0xffffffffu, best, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (ob > best || (ob == best && oi < bi)) {
                    best = ob;
                    bi = oi;
                }
            }
            if (bi != j && best > 0.f)
                for (int c = j + lane; c < cols; c += 32) {
                    const float a = W[j * ldw + c];
                    W[j * ldw + c] = W[bi * ldw + c];
                    W[bi * ldw + c] = a;
                }
        }
        __syncthreads();
        const float piv = W[j * ldw + j];
        if (!(fabsf(piv) > 0.f))
            return j + 1;
        const float ip = 1.f / piv;
        const int w = cols - j - 1;
        for (int e = threadIdx.x; e < n * w; e += blockDim.x) {
            const int i = e / w, c = j + 1 + e % w;
            if (i != j)
                W[i * ldw + c] = fmaf(-W[i * ldw + j] * ip, W[j * ldw + c], W[i * ldw + c]);
        }
    }
    __syncthreads();
    return 0;
}

// dst (n x n) <- symmetrised src; dst may be global or shared.
__device__ __forceinline__ void sym_store(int n, const float* src, float* dst)
{
    for (int e = threadIdx.x; e < n * n; e += blockDim.x) {
        const int i = e / n, j = e % n;
        dst[e] = 0.5f * (src[i * n + j] + src[j * n + i]);
    }
}

// Pout <- apply(e, Pin).  Pin in shared (sPin).  Uses W (n x 2n) and T (n x n).
// Result left symmetrised in sPout (shared).  Returns pivot failure code (uniform) or 0.
__device__ __forceinline__ int pair_apply(int n, const float* sAe, const float* sCe, const float* sJe,
                                          const float* sPin, float* sPout, float* W, float* T)
{
    const int ldw = 2 * n;
    // W = [I + Pin Ce | Pin Ae]
    smem_gemm<false>(n, n, n, sPin, n, sCe, n, W, ldw, nullptr, 0);
    smem_gemm<false>(n, n, n, sPin, n, sAe, n, W + n, ldw, nullptr, 0);
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x)
        W[i * ldw + i] += 1.f;
    const int bad = smem_gauss_jordan(n, n, W, ldw);
    if (bad)
        return bad;
    for (int e = threadIdx.x; e < n * n; e += blockDim.x) {
        const int i = e / n, c = e % n;
        T[e] = W[i * ldw + n + c] / W[i * ldw + i];
    }
    __syncthreads();
    smem_gemm<true>(n, n, n, sAe, n, T, n, W, n, sJe, n);      // W[0:n*n] = Je + Ae' X
    __syncthreads();
    sym_store(n, W, sPout);
    __syncthreads();
    return 0;
}

// e <- e o e (in place).  Uses W (n x 3n), T0, T1 (n x n).
__device__ __forceinline__ int pair_square(int n, float* sAe, float* sCe, float* sJe, float* W, float* T0,
                                           float* T1)
{
    const int ldw = 3 * n;
    // W = [I + Ce Je | Ae | Ce]
    smem_gemm<false>(n, n, n, sCe, n, sJe, n, W, ldw, nullptr, 0);
    for (int e = threadIdx.x; e < n * n; e += blockDim.x) {
        const int i = e / n, c = e % n;
        W[i * ldw + n + c] = sAe[e];
        W[i * ldw + 2 * n + c] = sCe[e];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x)
        W[i * ldw + i] += 1.f;
    const int bad = smem_gauss_jordan(n, 2 * n, W, ldw);
    if (bad)
        return bad;
    // T0 = XA = W Ae,  T1 = XC = W Ce   (W here is (I + Ce Je)^{-1})
    for (int e = threadIdx.x; e < n * n; e += blockDim.x) {
        const int i = e / n, c = e % n;
        const float d = 1.f / W[i * ldw + i];
        T0[e] = W[i * ldw + n + c] * d;
        T1[e] = W[i * ldw + 2 * n + c] * d;
    }
    __syncthreads();
    float* U0 = W;              // n x n temporaries inside W
    float* U1 = W + n * n;
    float* U2 = W + 2 * n * n;
    smem_gemm<false>(n, n, n, sJe, n, T0, n, U0, n, nullptr, 0);     // U0 = Je XA
    smem_gemm<false>(n, n, n, sAe, n, T1, n, U1, n, nullptr, 0);     // U1 = Ae XC
    __syncthreads();
    smem_gemm<true>(n, n, n, sAe, n, U0, n, U2, n, sJe, n);          // U2 = Je + Ae' Je XA  (new J)
    __syncthreads();
    sym_store(n, U2, sJe);
    // new C = U1 Ae' + Ce : (U1 Ae')[i][j] = sum_k U1[i][k] Ae[j][k]
    for (int e = threadIdx.x; e < n * n; e += blockDim.x) {
        const int i = e / n, j = e % n;
        float s = sCe[e];
        for (int k = 0; k < n; ++k)
            s = fmaf(U1[i * n + k], sAe[j * n + k], s);
        U0[e] = s;
    }
    __syncthreads();
    sym_store(n, U0, sCe);
    smem_gemm<false>(n, n, n, sAe, n, T0, n, U2, n, nullptr, 0);     // new A = Ae XA
    __syncthreads();
    for (int e = threadIdx.x; e < n * n; e += blockDim.x)
        sAe[e] = U2[e];
    __syncthreads();
    return 0;
}

inline size_t scan_smem_bytes(int n, int m)
{
    const int d = n > m ? n : m;
    // Ae, Ce, Je, Pcur, T0, T1: 6 d^2 ; W: 3 d^2 ; col: d
    return sizeof(float) * (size_t)(9 * d * d + d);
}

// Scan kernel: one CTA per instance.  pfull != 0: writes P_t, t = 0..H, to Pbuf [N][H+1][n][n].
// pfull == 0: writes only P_1 to Pbuf [N][n][n] (for H = 1, P_1 = Q).  Failures are recorded in
// fail_flag[inst] (0 = ok) for the gain/rollout kernel to act on.
__global__ void __launch_bounds__(256) scan_pair_kernel(SolveParams p, float* Pbuf, int* fail_flag, int pfull)
{
    extern __shared__ __align__(16) float sm[];
    const int n = p.n, m = p.m, H = p.H;
    const int d = n > m ? n : m;
    float* sAe = sm;
    float* sCe = sAe + d * d;
    float* sJe = sCe + d * d;
    float* sP = sJe + d * d;
    float* T0 = sP + d * d;
    float* T1 = T0 + d * d;
    float* W = T1 + d * d;
    float* scol = W + 3 * d * d;

    for (long long widx = blockIdx.x; widx < p.b0 * p.b1 * p.tcount; widx += gridDim.x) {
        const long long inst = window_instance(p, widx);
        __syncthreads();
        int fail = 0;
        // ---- step element: Ae = A, Je = Q, Ce = B R^{-1} B'
        load_to_smem(sAe, p.A, operand_offset(p.A, inst, p.b1, p.b2), n * n);
        load_to_smem(sJe, p.Q, operand_offset(p.Q, inst, p.b1, p.b2), n * n);
        load_to_smem(T0, p.R, operand_offset(p.R, inst, p.b1, p.b2), m * m);
        load_to_smem(T1, p.B, operand_offset(p.B, inst, p.b1, p.b2), n * m);
        __syncthreads();
        for (int e = threadIdx.x; e < m * n; e += blockDim.x)   // W = B' (m x n)
            W[e] = T1[(e % n) * m + e / n];
        const int badR = smem_cholesky(m, T0, scol);
        if (badR) {
            fail = (H - 1) * m + badR;   // R itself is not PD: the first step (t = H-1) fails
        } else {
            smem_chol_solve_neg(m, n, T0, W);                   // W = -R^{-1} B'
            __syncthreads();
            smem_gemm<false>(n, n, m, T1, m, W, n, sCe, n, nullptr, 0);
            __syncthreads();
            for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                sCe[e] = -sCe[e];
            __syncthreads();
            sym_store(n, sCe, T0);
            __syncthreads();
            for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                sCe[e] = T0[e];
            __syncthreads();
        }

        if (!fail && pfull) {
            float* Pi = Pbuf + inst * (long long)(H + 1) * n * n;
            for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                Pi[(long long)H * n * n + e] = sJe[e];          // P_H = Q
            __syncthreads();
            for (int step = 1; step <= H && !fail; step <<= 1) {
                const int kend = min(2 * step - 1, H);
                for (int k = step; k <= kend && !fail; ++k) {
                    const float* src = Pi + (long long)(H - k + step) * n * n;
                    for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                        sP[e] = src[e];
                    __syncthreads();
                    const int bad = pair_apply(n, sAe, sCe, sJe, sP, T0, W, T1);
                    if (bad) {
                        fail = (H - k) * m + 1;
                        break;
                    }
                    float* dst = Pi + (long long)(H - k) * n * n;
                    for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                        dst[e] = T0[e];
                    __syncthreads();
                }
                if (!fail && 2 * step <= H) {
                    const int bad = pair_square(n, sAe, sCe, sJe, W, T0, T1);
                    if (bad)
                        fail = 1;
                }
            }
        } else if (!fail) {
            // P_1 = apply(e^(H-1), Q): binary digits of H-1, squaring as we go
            for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                sP[e] = sJe[e];
            __syncthreads();
            int rem = H - 1;
            while (rem > 0 && !fail) {
                if (rem & 1) {
                    const int bad = pair_apply(n, sAe, sCe, sJe, sP, T0, W, T1);
                    if (bad) {
                        fail = 1;
                        break;
                    }
                    for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                        sP[e] = T0[e];
                    __syncthreads();
                }
                rem >>= 1;
                if (rem > 0) {
                    const int bad = pair_square(n, sAe, sCe, sJe, W, T0, T1);
                    if (bad)
                        fail = 1;
                }
            }
            if (!fail) {
                float* dst = Pbuf + inst * (long long)n * n;
                for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                    dst[e] = sP[e];
            }
        }
        if (threadIdx.x == 0)
            fail_flag[inst] = fail;
    }
}

inline size_t gain_rollout_smem_bytes(int n, int m)
{
    return riccati_cta_smem_bytes(n, m);
}

// Fused gain + forward rollout (Eq. 4 of Prop. 3.1 and the second loop of Alg. 1), forward in
// time: K_t from P_{t+1}, u_t = K_t x_t, x_{t+1} = A x_t + B u_t.  One CTA per instance.
// pfull != 0: Pbuf = [N][H+1][n][n] holds every P_t (it may be the caller's P).
// pfull == 0: Pbuf = [N][n][n] holds P_1; only t = 0 is processed and the kernel also forms
// P_0 = Q + A'P_1 A + Y'K_0 and writes it to p.P.
__global__ void __launch_bounds__(256) gain_rollout_kernel(SolveParams p, const float* Pbuf,
                                                           const int* fail_flag, int pfull)
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
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;

    for (long long widx = blockIdx.x; widx < p.b0 * p.b1 * p.tcount; widx += gridDim.x) {
        const long long inst = window_instance(p, widx);
        __syncthreads();
        int fail = fail_flag ? fail_flag[inst] : 0;
        if (fail) {
            cta_fail_instance(p, inst, fail);
            continue;
        }
        float* xo = p.x ? p.x + inst * (long long)(H + 1) * n : nullptr;
        float* uo = p.u ? p.u + inst * (long long)(p.first_only ? m : H * m) : nullptr;
        float* Ko = p.K ? p.K + inst * (long long)H * m * n : nullptr;
        const bool roll = (xo != nullptr) || (uo != nullptr);
        const bool want_p0 = !pfull && p.P != nullptr;
        int steps = 0;
        if (Ko || xo || (uo && !p.first_only))
            steps = H;
        else if (uo || want_p0)
            steps = 1;
        if (!pfull)
            steps = min(steps, 1);
        if (pfull && p.first_only && p.P) {            // P_0 only: copy it out of the full buffer
            const float* src = Pbuf + inst * (long long)(H + 1) * n * n;
            float* dst = p.P + inst * (long long)n * n;
            for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                dst[e] = src[e];
        }
        if (steps > 0) {
            load_to_smem(sA, p.A, operand_offset(p.A, inst, p.b1, p.b2), n * n);
            load_to_smem(sB, p.B, operand_offset(p.B, inst, p.b1, p.b2), n * m);
            load_to_smem(sR, p.R, operand_offset(p.R, inst, p.b1, p.b2), m * m);
            load_to_smem(sQ, p.Q, operand_offset(p.Q, inst, p.b1, p.b2), n * n);
            if (p.x0.ptr)
                load_to_smem(sx, p.x0, operand_offset(p.x0, inst, p.b1, p.b2), n);
            __syncthreads();
            if (xo)
                for (int e = threadIdx.x; e < n; e += blockDim.x)
                    xo[e] = sx[e];
        }
        for (int t = 0; t < steps; ++t) {
            const float* src = pfull ? Pbuf + (inst * (long long)(H + 1) + t + 1) * n * n
                                     : Pbuf + inst * (long long)n * n;
            for (int e = threadIdx.x; e < n * n; e += blockDim.x)
                sP[e] = src[e];
            __syncthreads();
            smem_gemm<false>(n, m, n, sP, n, sB, m, sV, m, nullptr, 0);
            smem_gemm<false>(n, n, n, sP, n, sA, n, sT, n, nullptr, 0);
            __syncthreads();
            smem_gemm<true>(m, m, n, sB, m, sV, m, sS, m, sR, m);
            smem_gemm<true>(m, n, n, sB, m, sT, n, sY, n, nullptr, 0);
            __syncthreads();
            const int bad = smem_cholesky(m, sS, scol);
            if (bad) {
                fail = t * m + bad;
                break;
            }
            for (int e = threadIdx.x; e < m * n; e += blockDim.x)
                sK[e] = sY[e];
            __syncthreads();
            smem_chol_solve_neg(m, n, sS, sK);
            __syncthreads();
            if (Ko)
                for (int e = threadIdx.x; e < m * n; e += blockDim.x)
                    Ko[(long long)t * m * n + e] = sK[e];
            if (want_p0) {
                smem_gemm<true>(n, n, n, sA, n, sT, n, sP, n, sQ, n);
                __syncthreads();
                smem_gemm<true>(n, n, m, sY, n, sK, n, sP, n, sP, n);
                __syncthreads();
                sym_store(n, sP, p.P + inst * (long long)n * n);
            }
            if (roll) {
                for (int i = warp; i < m; i += nw) {
                    const float s = warp_dot(sK + i * n, sx, n);
                    if (lane == 0)
                        su[i] = s;
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
            }
            __syncthreads();
        }
        if (fail) {
            __syncthreads();
            cta_fail_instance(p, inst, fail);
        } else if (p.info && threadIdx.x == 0) {
            p.info[inst] = 0;
        }
    }
}

// Enqueue the scan path: scan kernel (value matrices) then the gain/rollout kernel.
inline cudaError_t launch_scan_path(const SolveParams& p, float* Pbuf, int* fail_flag, int pfull, int sm_count,
                                    cudaStream_t st, int* launches)
{
    cudaError_t e;
    const size_t sm1 = scan_smem_bytes(p.n, p.m), sm2 = gain_rollout_smem_bytes(p.n, p.m);
    if ((e = cudaFuncSetAttribute(scan_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm1)))
        return e;
    if ((e = cudaFuncSetAttribute(gain_rollout_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm2)))
        return e;
    int o1 = 1, o2 = 1;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o1, scan_pair_kernel, 256, sm1))) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o2, gain_rollout_kernel, 256, sm2))) return e;
    long long g1 = (long long)sm_count * (o1 < 1 ? 1 : o1), g2 = (long long)sm_count * (o2 < 1 ? 1 : o2);
    const long long nwin = p.b0 * p.b1 * p.tcount;
    if (g1 > nwin) g1 = nwin;
    if (g2 > nwin) g2 = nwin;
    scan_pair_kernel<<<(unsigned)g1, 256, sm1, st>>>(p, Pbuf, fail_flag, pfull);
    if ((e = cudaGetLastError())) return e;
    gain_rollout_kernel<<<(unsigned)g2, 256, sm2, st>>>(p, Pbuf, fail_flag, pfull);
    if ((e = cudaGetLastError())) return e;
    *launches = 2;
    return cudaSuccess;
}

} // namespace ttc
