// Symplectic-pair scan over the horizon for n = m = 16 / 32, parallel in time (time-invariant problems).
//
// Element of the scan: the symplectic transition matrix of Thm A.2 kept inverse-free as e = (A, C, J) (C = B R^{-1} B',
// J = Q for one step) together with a factor G of C = G G'.  With that factor both operations of the scan are
// Riccati-type steps whose only solve is a Cholesky factorisation of a matrix I + G'(.)G >= I:
//     apply(e, P)  = J + A'P A - Y'S^{-1}Y,   S = I + G'P G,  Y = G'P A            (Prop. 3.1 with B = G, R = I, Q = J)
//     e o e        : Jt = J - J G S^{-1} G'J  (S = I + G'J G),   W = I - C Jt = (I + C J)^{-1},
//                    A2 = A W A,   C2 = C + A (C - C Jt C) A',   J2 = J + A'Jt A,   G2 = chol(C2).
// The problem is time-invariant, so the suffix products are powers: round r holds e^(2^r) and produces
// P_{H-k} = apply(e^(2^r), P_{H-k+2^r}) for 2^r <= k < 2^(r+1).  All applications of a round, over all instances, are
// independent work items of ONE launch (scan_step_kernel), the squarings of a round are another
// (scan_square_kernel): the depth over the horizon is 2 log2(H) launches instead of H dependent steps.
// Afterwards every gain K_t = -(R + B'P_{t+1}B)^{-1} B'P_{t+1}A is again one independent item per (instance, t)
// (scan_step_kernel in its gain form), and scan_rollout_kernel runs the forward loop of Alg. 1.
//
// Thread mapping as in riccati_warp.cuh: N lanes own one item, lane c holds column c of every matrix in registers;
// symmetric matrices are read by rows as columns; cross-lane traffic is broadcast reads of shared-memory rows.
#pragma once

#include "common.cuh"
#include "riccati_warp.cuh"

namespace ttc {
namespace scanw {

using rwarp::Shape;
using rwarp::f32x2;
using rwarp::load_row;
using rwarp::store_row;
using rwarp::pack_row;
using rwarp::unpack_row;
using rwarp::axpy_row;

constexpr int WARPS = rwarp::WARPS;
constexpr int THREADS = rwarp::THREADS;
constexpr int ELEM_MATS = 4;                    // A | C | G | J per instance in the element workspace

// out[:] += sum_k coef[k] * row_k(M)      (M row-major in shared memory, row stride LD)
template <int N>
__device__ __forceinline__ void mix(f32x2 (&out)[N / 2], const float (&coef)[N], const float* M)
{
#pragma unroll
    for (int k = 0; k < N; ++k)
        axpy_row<N>(out, coef[k], M + k * Shape<N>::LD);
}
template <int N>
__device__ __forceinline__ void zero2(f32x2 (&v)[N / 2])
{
#pragma unroll
    for (int i = 0; i < N / 2; ++i)
        v[i] = 0ull;
}
template <int N>
__device__ __forceinline__ void load_col(float (&v)[N], const float* M, int c)
{
#pragma unroll
    for (int k = 0; k < N; ++k)
        v[k] = M[k * Shape<N>::LD + c];
}
template <int N>
__device__ __forceinline__ void store_col(float* M, int c, const float (&v)[N])
{
#pragma unroll
    for (int k = 0; k < N; ++k)
        M[k * Shape<N>::LD + c] = v[k];
}
// matrix (row-major, dense, N x N floats in global memory) -> shared memory rows; lane c takes column c of every row
template <int N>
__device__ __forceinline__ void load_matrix(float* dst, const float* src, int c)
{
#pragma unroll 8
    for (int k = 0; k < N; ++k)
        dst[k * Shape<N>::LD + c] = __ldg(src + k * N + c);
}

// Cholesky of a symmetric positive SEMI-definite matrix spread over N lanes (lane c = row c): a pivot that is not
// larger than `tiny` gives a zero column (the matrix has no weight in that direction).  On return s = row c of the
// factor, zero right of the diagonal.  Never fails; NaN input gives NaN output.
template <int N>
__device__ __forceinline__ void seg_chol_psd(float (&s)[N], int c, float tiny)
{
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const float sj = s[j];
        const float d = __shfl_sync(0xffffffffu, sj, j, N);
        const bool ok = d > tiny;
        const float rinv = ok ? __frcp_rn(d) : 0.f;
        const float f = sj * rinv;
#pragma unroll
        for (int cc = j + 1; cc < N; ++cc) {
            const float lc = __shfl_sync(0xffffffffu, sj, cc, N);
            s[cc] = fmaf(-f, lc, s[cc]);
        }
        s[j] = (ok && j <= c) ? sj * rsqrtf(d) : 0.f;
    }
}

// y <- L^{-1} y with the rows of L' (columns of L) broadcast from Lt and the reciprocal pivots in rinv
template <int N>
__device__ __forceinline__ void forward_subst(float (&y)[N], const float* Lt, const float (&rinv)[N])
{
    constexpr int LD = Shape<N>::LD;
#pragma unroll
    for (int k = 0; k < N; ++k) {
        const float zk = y[k] * rinv[k];
        y[k] = zk;
        const float* lt = Lt + k * LD;
#pragma unroll
        for (int i4 = (k + 1) & ~3; i4 < N; i4 += 4) {
            const float4 l4 = *reinterpret_cast<const float4*>(lt + i4);
            if (i4 + 0 > k) y[i4 + 0] = fmaf(-l4.x, zk, y[i4 + 0]);
            if (i4 + 1 > k) y[i4 + 1] = fmaf(-l4.y, zk, y[i4 + 1]);
            if (i4 + 2 > k) y[i4 + 2] = fmaf(-l4.z, zk, y[i4 + 2]);
            if (i4 + 3 > k) y[i4 + 3] = fmaf(-l4.w, zk, y[i4 + 3]);
        }
    }
}
// y <- L^{-T} y with the rows of L broadcast from Ls
template <int N>
__device__ __forceinline__ void backward_subst(float (&y)[N], const float* Ls, const float (&rinv)[N])
{
    constexpr int LD = Shape<N>::LD;
#pragma unroll
    for (int k = N - 1; k >= 0; --k) {
        const float xk = y[k] * rinv[k];
        y[k] = xk;
        const float* lr = Ls + k * LD;
#pragma unroll
        for (int i4 = 0; i4 < k; i4 += 4) {
            const float4 l4 = *reinterpret_cast<const float4*>(lr + i4);
            if (i4 + 0 < k) y[i4 + 0] = fmaf(-l4.x, xk, y[i4 + 0]);
            if (i4 + 1 < k) y[i4 + 1] = fmaf(-l4.y, xk, y[i4 + 1]);
            if (i4 + 2 < k) y[i4 + 2] = fmaf(-l4.z, xk, y[i4 + 2]);
            if (i4 + 3 < k) y[i4 + 3] = fmaf(-l4.w, xk, y[i4 + 3]);
        }
    }
}
// factor rows -> L (rows), Lt (rows of L'), rinv; the caller synchronises the warp before and after
template <int N>
__device__ __forceinline__ void publish_factor(float* Ls, float* Lt, float* rinv_s, const float (&s)[N], float rs_own, int c)
{
    store_row<N>(Ls + c * Shape<N>::LD, s);
    store_col<N>(Lt, c, s);
    rinv_s[c] = rs_own;
}
__device__ __forceinline__ void record_failure(int* fail_flag, long long inst, int code)
{
    atomicCAS(fail_flag + inst, 0, code);
}

struct ScanParams {
    SolveParams sp;
    float* elem;        // [N][4][n][n]: A_e | C_e | G_e | J_e of the current power of the step element
    float* Pbuf;        // [N][H+1][n][n]: every P_t (the caller's P or workspace)
    int* fail_flag;     // [N]: 0, or a positive code once something failed for the instance
    int step;           // apply form: 2^r
    int cnt;            // apply form: applications per instance in this round
    int gain_steps;     // gain form: gains per instance (H, or 1 when only u_0 is wanted)
};

// ---- element of one step: A, C = B R^{-1} B', G = B L_R^{-T} (R = L_R L_R'), J = Q; also P_H = Q ------------------------
template <int N>
struct InitSlot {
    float B[Shape<N>::MAT], G[Shape<N>::MAT], L[Shape<N>::MAT], Lt[Shape<N>::MAT], rinv[N];
};
template <int N>
__global__ void __launch_bounds__(THREADS) scan_init_kernel(ScanParams q)
{
    using S = Shape<N>;
    constexpr int LD = S::LD;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const SolveParams& p = q.sp;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, sub = lane / N, c = lane % N;
    InitSlot<N>& sl = reinterpret_cast<InitSlot<N>*>(smem_raw)[warp * S::IPW + sub];
    const long long nwin = p.b0 * p.b1 * p.tcount;
    const int H = p.H;
    for (long long base = (long long)blockIdx.x * S::SLOTS; base < nwin; base += (long long)gridDim.x * S::SLOTS) {
        const long long w = base + warp * S::IPW + sub;
        const bool active = w < nwin;
        const long long inst = window_instance(p, active ? w : base);
        const float* Ag = reinterpret_cast<const float*>(p.A.ptr) + operand_offset(p.A, inst, p.b1, p.b2);
        const float* Bg = reinterpret_cast<const float*>(p.B.ptr) + operand_offset(p.B, inst, p.b1, p.b2);
        const float* Rg = reinterpret_cast<const float*>(p.R.ptr) + operand_offset(p.R, inst, p.b1, p.b2);
        const long long oq = operand_offset(p.Q, inst, p.b1, p.b2);
        float* E = q.elem + inst * (long long)(ELEM_MATS * N * N);
        __syncwarp();
        load_matrix<N>(sl.B, Bg, c);
        float s[N];
#pragma unroll
        for (int l = 0; l < N; ++l)
            s[l] = __ldg(Rg + c * N + l);                      // row c of R
        float rs_own;
        const int bad = rwarp::seg_chol<N>(s, rs_own, c);
        if (bad && active && c == 0)
            record_failure(q.fail_flag, inst, (H - 1) * N + bad);      // R itself is not positive definite
        publish_factor<N>(sl.L, sl.Lt, sl.rinv, s, rs_own, c);
        __syncwarp();
        float rinv[N], g[N];
        load_row<N>(rinv, sl.rinv);
        load_row<N>(g, sl.B + c * LD);                         // row c of B
        forward_subst<N>(g, sl.Lt, rinv);                      // row c of G = B L_R^{-T}
        store_col<N>(sl.G, c, g);                              // rows of G' (columns of G)
        __syncwarp();
        f32x2 c2[N / 2];
        zero2<N>(c2);
        mix<N>(c2, g, sl.G);                                   // row c of C = G G'
        float crow[N];
        unpack_row<N>(crow, c2);
        if (active) {
#pragma unroll
            for (int l = 0; l < N; ++l) {
                const float a = __ldg(Ag + c * N + l);
                const float qv = load_elem(p.Q, oq + c * N + l);
                E[0 * N * N + c * N + l] = a;
                E[1 * N * N + c * N + l] = crow[l];
                E[2 * N * N + c * N + l] = g[l];
                E[3 * N * N + c * N + l] = qv;
                q.Pbuf[(inst * (long long)(H + 1) + H) * N * N + c * N + l] = qv;      // P_H = Q
            }
        }
    }
}

// ---- one Riccati-type step per work item ---------------------------------------------------------------------------
// GAIN = false: item (instance, j): P_{H-k} = apply(e, P_{H-k+step}), k = step + j, operands from the element workspace.
// GAIN = true : item (instance, t): K_t = -(R + B'P_{t+1}B)^{-1} B'P_{t+1}A with the problem's own A, B, R.
template <int N>
struct StepSlot {
    float A[Shape<N>::MAT], B[Shape<N>::MAT];
    float buf0[Shape<N>::MAT];     // rows of P, then rows of Z
    float L[Shape<N>::MAT], Lt[Shape<N>::MAT];
    float rinv[N];
};
template <int N, bool GAIN>
__global__ void __launch_bounds__(THREADS, (N == 32) ? 2 : 3) scan_step_kernel(ScanParams q)
{
    using S = Shape<N>;
    constexpr int LD = S::LD;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const SolveParams& p = q.sp;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, sub = lane / N, c = lane % N;
    StepSlot<N>& sl = reinterpret_cast<StepSlot<N>*>(smem_raw)[warp * S::IPW + sub];
    const int H = p.H;
    const long long per = GAIN ? q.gain_steps : q.cnt;
    const long long nitems = p.b0 * p.b1 * p.tcount * per;
    for (long long base = (long long)blockIdx.x * S::SLOTS; base < nitems; base += (long long)gridDim.x * S::SLOTS) {
        const long long it = base + warp * S::IPW + sub;
        const bool active = it < nitems;
        const long long itv = active ? it : base;
        const long long inst = window_instance(p, itv / per);
        const int j = (int)(itv % per);
        const float *Ag, *Bg, *Pin;
        float* E = q.elem + inst * (long long)(ELEM_MATS * N * N);
        int tout;                                              // time index of the result
        if (GAIN) {
            Ag = reinterpret_cast<const float*>(p.A.ptr) + operand_offset(p.A, inst, p.b1, p.b2);
            Bg = reinterpret_cast<const float*>(p.B.ptr) + operand_offset(p.B, inst, p.b1, p.b2);
            tout = j;
            Pin = q.Pbuf + (inst * (long long)(H + 1) + j + 1) * N * N;
        } else {
            Ag = E;
            Bg = E + 2 * N * N;
            const int k = q.step + j;
            tout = H - k;
            Pin = q.Pbuf + (inst * (long long)(H + 1) + H - k + q.step) * N * N;
        }
        __syncwarp();                                          // the previous item's reads of the slot are done
        load_matrix<N>(sl.A, Ag, c);
        load_matrix<N>(sl.B, Bg, c);
        load_matrix<N>(sl.buf0, Pin, c);
        float s[N];                                            // column c of R (identity for an element), then of S
        if (GAIN) {
            const float* Rg = reinterpret_cast<const float*>(p.R.ptr) + operand_offset(p.R, inst, p.b1, p.b2);
#pragma unroll
            for (int l = 0; l < N; ++l)
                s[l] = __ldg(Rg + c * N + l);
        } else {
#pragma unroll
            for (int l = 0; l < N; ++l)
                s[l] = (l == c) ? 1.f : 0.f;
        }
        __syncwarp();
        float y[N];
        f32x2 p2[N / 2];
        float pn[N];                                           // tensor-core path: column c of J + A'T
        // n = 32: the dense products run on the tensor cores (three-pass tf32 mma.sync, rwarp::mma32_product), one copy
        // of the product code in phases as in riccati_warp_kernel: V = P B -> L, T = P A -> L', B'V -> buf0, Y = B'T -> L,
        // A'T -> L' (applications only); the last phase factorises, substitutes and, for an application, runs Z'Z -> L.
        constexpr bool MMA = (N == 32);
        constexpr int LAST = GAIN ? 4 : 5;
#pragma unroll 1
        for (int ph = MMA ? 0 : LAST; ph <= LAST; ++ph) {
        if (!MMA || ph == LAST) {
        if constexpr (MMA) {
            float tmp[N];
            load_row<N>(tmp, sl.buf0 + c * LD);                // (B'V)[c,:] = (B'V)[:,c]
#pragma unroll
            for (int l = 0; l < N; ++l) {
                s[l] += tmp[l];
                y[l] = sl.L[l * LD + c];
            }
            if (!GAIN) {
#pragma unroll
                for (int l = 0; l < N; ++l)
                    pn[l] = __ldg(E + 3 * N * N + c * N + l) + sl.Lt[l * LD + c];
            }
        } else {
            // The dense loops run over k with four-fold unrolling and take their coefficients from the lane's own column
            // of a shared-memory matrix (a fully unrolled body would be bound by instruction fetch).
            {
                f32x2 v2[N / 2], t2[N / 2];
                zero2<N>(v2);
                zero2<N>(t2);
#pragma unroll 4
                for (int i = 0; i < N; ++i) {                      // V[:,c] = P B[:,c], T[:,c] = P A[:,c]
                    const float bic = sl.B[i * LD + c], aic = sl.A[i * LD + c];
                    const f32x2 b2 = rwarp::pack2(bic, bic), a2 = rwarp::pack2(aic, aic);
                    const float* prow = sl.buf0 + i * LD;
#pragma unroll
                    for (int q4 = 0; q4 < N / 4; ++q4) {
                        const ulonglong2 t4 = *reinterpret_cast<const ulonglong2*>(prow + 4 * q4);
                        rwarp::fma2(v2[2 * q4], t4.x, b2);
                        rwarp::fma2(v2[2 * q4 + 1], t4.y, b2);
                        rwarp::fma2(t2[2 * q4], t4.x, a2);
                        rwarp::fma2(t2[2 * q4 + 1], t4.y, a2);
                    }
                }
                float v[N], t[N];
                unpack_row<N>(v, v2);
                unpack_row<N>(t, t2);
                store_col<N>(sl.L, c, v);                          // own column only: no exchange
                store_col<N>(sl.Lt, c, t);
            }
            {
                f32x2 s2[N / 2], y2[N / 2];
                pack_row<N>(s2, s);
                zero2<N>(y2);
                if (!GAIN) {
                    float jc[N];
#pragma unroll
                    for (int l = 0; l < N; ++l)
                        jc[l] = __ldg(E + 3 * N * N + c * N + l);  // row c of J = column c
                    pack_row<N>(p2, jc);
                }
#pragma unroll 4
                for (int k = 0; k < N; ++k) {                      // S += B'V, Y = B'T, Pn = J + A'T: each row read once
                    const float vk = sl.L[k * LD + c], tk = sl.Lt[k * LD + c];
                    const f32x2 vv = rwarp::pack2(vk, vk), tt = rwarp::pack2(tk, tk);
#pragma unroll
                    for (int q4 = 0; q4 < N / 4; ++q4) {
                        const ulonglong2 b4 = *reinterpret_cast<const ulonglong2*>(sl.B + k * LD + 4 * q4);
                        rwarp::fma2(s2[2 * q4], vv, b4.x);
                        rwarp::fma2(s2[2 * q4 + 1], vv, b4.y);
                        rwarp::fma2(y2[2 * q4], tt, b4.x);
                        rwarp::fma2(y2[2 * q4 + 1], tt, b4.y);
                        if (!GAIN) {
                            const ulonglong2 a4 = *reinterpret_cast<const ulonglong2*>(sl.A + k * LD + 4 * q4);
                            rwarp::fma2(p2[2 * q4], tt, a4.x);
                            rwarp::fma2(p2[2 * q4 + 1], tt, a4.y);
                        }
                    }
                }
                unpack_row<N>(s, s2);
                unpack_row<N>(y, y2);
            }
        }
        float rs_own;
        const int bad = rwarp::seg_chol<N>(s, rs_own, c);
        if (bad && active && c == 0)
            record_failure(q.fail_flag, inst, tout * N + bad);
        __syncwarp();                                          // every lane is done with the rows of P
        publish_factor<N>(sl.L, sl.Lt, sl.rinv, s, rs_own, c);
        __syncwarp();
        float rinv[N];
        load_row<N>(rinv, sl.rinv);
        forward_subst<N>(y, sl.Lt, rinv);                      // Z[:,c] = L^{-1} Y[:,c]
        if (GAIN) {
            backward_subst<N>(y, sl.L, rinv);                  // -K[:,c] = L^{-T} Z[:,c]
            if (active && p.K) {
                float* kt = p.K + (inst * (long long)H + tout) * N * N + c;
#pragma unroll
                for (int l = 0; l < N; ++l)
                    kt[l * N] = -y[l];
            } else if (active) {
                float* kt = p.Kws + (inst * (long long)H + tout) * N * N + c;
#pragma unroll
                for (int l = 0; l < N; ++l)
                    kt[l * N] = -y[l];
            }
        } else {
            store_col<N>(sl.buf0, c, y);                       // rows of Z
            __syncwarp();
            float pcol[N];
            if constexpr (MMA) {
                float acc[2][4][4];
                rwarp::mma32_zero(acc);
                rwarp::mma32_product(acc, sl.buf0, sl.buf0, lane);
                rwarp::mma32_store(sl.L, acc, lane);           // nobody reads the rows of L in this form
                __syncwarp();
#pragma unroll
                for (int l = 0; l < N; ++l)
                    pcol[l] = pn[l] - sl.L[l * LD + c];        // Pn[:,c] - Z'Z[:,c]
            } else {
#pragma unroll 4
                for (int k = 0; k < N; ++k)                    // Pn[:,c] -= Z'Z[:,c]
                    axpy_row<N>(p2, -sl.buf0[k * LD + c], sl.buf0 + k * LD);
                unpack_row<N>(pcol, p2);
            }
            __syncwarp();
            store_row<N>(sl.buf0 + c * LD, pcol);              // column c as row c, then average with the transpose
            __syncwarp();
#pragma unroll
            for (int l = 0; l < N; ++l)
                pcol[l] = 0.5f * (pcol[l] + sl.buf0[l * LD + c]);
            if (active) {
                float4* dst = reinterpret_cast<float4*>(q.Pbuf + (inst * (long long)(H + 1) + tout) * N * N + c * N);
#pragma unroll
                for (int l4 = 0; l4 < N / 4; ++l4)
                    dst[l4] = make_float4(pcol[4 * l4], pcol[4 * l4 + 1], pcol[4 * l4 + 2], pcol[4 * l4 + 3]);
            }
        }
        } else if constexpr (MMA) {
            // phase:  0      1      2      3      4
            // A'   :  P      P      B'     B'     A'          (P symmetric, so P B = P'B)
            // B    :  B      A      V      T      T
            // to   :  L      L'     buf0   L      L'          (buf0: P, then B'V)
            const float* Am = ph < 2 ? sl.buf0 : ph == 4 ? sl.A : sl.B;
            const float* Bm = ph == 0 ? sl.B : ph == 1 ? sl.A : ph == 2 ? sl.L : sl.Lt;
            float* Dm = ph == 1 || ph == 4 ? sl.Lt : ph == 2 ? sl.buf0 : sl.L;
            float acc[2][4][4];
            rwarp::mma32_zero(acc);
            rwarp::mma32_product(acc, Am, Bm, lane);
            __syncwarp();                                      // every lane has read what the result overwrites
            rwarp::mma32_store(Dm, acc, lane);
            __syncwarp();
        }
        }                                                      // phases
    }
}

// ---- e <- e o e, one instance per slot ---------------------------------------------------------------------------------
template <int N>
struct SquareSlot {
    float A[Shape<N>::MAT], C[Shape<N>::MAT], G[Shape<N>::MAT], J[Shape<N>::MAT];
    float T0[Shape<N>::MAT], T1[Shape<N>::MAT], T2[Shape<N>::MAT];
    float L[Shape<N>::MAT], Lt[Shape<N>::MAT];
    float rinv[N];
};
template <int N>
__global__ void __launch_bounds__(THREADS, 1) scan_square_kernel(ScanParams q)
{
    using S = Shape<N>;
    constexpr int LD = S::LD;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const SolveParams& p = q.sp;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, sub = lane / N, c = lane % N;
    SquareSlot<N>& sl = reinterpret_cast<SquareSlot<N>*>(smem_raw)[warp * S::IPW + sub];
    const long long nwin = p.b0 * p.b1 * p.tcount;
    for (long long base = (long long)blockIdx.x * S::SLOTS; base < nwin; base += (long long)gridDim.x * S::SLOTS) {
        const long long w = base + warp * S::IPW + sub;
        const bool active = w < nwin;
        const long long inst = window_instance(p, active ? w : base);
        float* E = q.elem + inst * (long long)(ELEM_MATS * N * N);
        __syncwarp();
        load_matrix<N>(sl.A, E, c);
        load_matrix<N>(sl.C, E + N * N, c);
        load_matrix<N>(sl.G, E + 2 * N * N, c);
        load_matrix<N>(sl.J, E + 3 * N * N, c);
        __syncwarp();
        float jc[N], t[N], vt[N], y[N], s[N];
        load_row<N>(jc, sl.J + c * LD);                        // column c of J (= row c)
        {
            float ac[N], gc[N], v[N];
            load_col<N>(ac, sl.A, c);
            load_col<N>(gc, sl.G, c);
            f32x2 a2[N / 2], b2[N / 2], c2[N / 2];
            zero2<N>(a2); zero2<N>(b2); zero2<N>(c2);
            mix<N>(a2, ac, sl.J);                              // T[:,c] = J A[:,c]
            mix<N>(b2, gc, sl.J);                              // V[:,c] = J G[:,c]
            mix<N>(c2, jc, sl.G);                              // (G'J)[:,c]
            unpack_row<N>(t, a2);
            unpack_row<N>(v, b2);
            unpack_row<N>(vt, c2);
            f32x2 s2[N / 2], y2[N / 2];
#pragma unroll
            for (int l = 0; l < N; ++l)
                s[l] = (l == c) ? 1.f : 0.f;
            pack_row<N>(s2, s);
            zero2<N>(y2);
            mix<N>(s2, v, sl.G);                               // S[:,c] = e_c + G'V[:,c]
            mix<N>(y2, t, sl.G);                               // Y[:,c] = G'T[:,c]
            unpack_row<N>(s, s2);
            unpack_row<N>(y, y2);
        }
        float rs_own;
        const int bad = rwarp::seg_chol<N>(s, rs_own, c);
        if (bad && active && c == 0)
            record_failure(q.fail_flag, inst, bad);
        publish_factor<N>(sl.L, sl.Lt, sl.rinv, s, rs_own, c);
        __syncwarp();
        float rinv[N];
        load_row<N>(rinv, sl.rinv);
        forward_subst<N>(y, sl.Lt, rinv);                      // Z[:,c]  = L^{-1} Y[:,c]
        forward_subst<N>(vt, sl.Lt, rinv);                     // U'[:,c] = L^{-1} (G'J)[:,c]
        store_col<N>(sl.T0, c, y);                             // rows of Z
        store_col<N>(sl.T1, c, vt);                            // rows of U'
        __syncwarp();
        float x[N], j2[N];
        {
            float zn[N], un[N];
#pragma unroll
            for (int l = 0; l < N; ++l) {
                zn[l] = -y[l];
                un[l] = -vt[l];
            }
            f32x2 jt2[N / 2], x2[N / 2], jn2[N / 2];
            pack_row<N>(jt2, jc);
            mix<N>(jt2, un, sl.T1);                            // Jt[:,c] = J[:,c] - U U'[:,c]     ((I + J C)^{-1} J)
            pack_row<N>(x2, t);
            mix<N>(x2, zn, sl.T1);                             // X[:,c] = (Jt A)[:,c] = T[:,c] - U Z[:,c]
            pack_row<N>(jn2, jc);
            mix<N>(jn2, t, sl.A);                              // J2[:,c] = J[:,c] + A'T[:,c] - Z'Z[:,c]
            mix<N>(jn2, zn, sl.T0);
            float jt[N];
            unpack_row<N>(jt, jt2);
            unpack_row<N>(x, x2);
            unpack_row<N>(j2, jn2);
            store_row<N>(sl.T2 + c * LD, jt);                  // rows of Jt (symmetric: column c = row c)
        }
        __syncwarp();                                          // Z, U' consumed; Jt visible
        float arow[N], a2row[N], c2row[N];
        load_row<N>(arow, sl.A + c * LD);
        {
            f32x2 d2[N / 2], f2[N / 2];
            float ac[N], cc[N];
            load_col<N>(ac, sl.A, c);
            load_row<N>(cc, sl.C + c * LD);                    // column c of C (= row c)
            float xn[N];
#pragma unroll
            for (int l = 0; l < N; ++l)
                xn[l] = -x[l];
            pack_row<N>(d2, ac);
            mix<N>(d2, xn, sl.C);                              // D[:,c] = A[:,c] - C X[:,c]      (D = (I + C J)^{-1} A)
            zero2<N>(f2);
            mix<N>(f2, cc, sl.T2);                             // F[:,c] = Jt C[:,c]
            float d[N], f[N];
            unpack_row<N>(d, d2);
            unpack_row<N>(f, f2);
            store_col<N>(sl.T0, c, d);                         // rows of D
            f32x2 e2[N / 2];
            pack_row<N>(e2, cc);
#pragma unroll
            for (int l = 0; l < N; ++l)
                f[l] = -f[l];
            mix<N>(e2, f, sl.C);                               // E[:,c] = C[:,c] - C F[:,c]      (E = (I + C J)^{-1} C, symmetric)
            float e[N];
            unpack_row<N>(e, e2);
            store_row<N>(sl.T1 + c * LD, e);                   // rows of E
        }
        __syncwarp();
        {
            f32x2 r2[N / 2], m2[N / 2];
            zero2<N>(r2);
            mix<N>(r2, arow, sl.T0);                           // row c of A2 = A D
            unpack_row<N>(a2row, r2);
            zero2<N>(m2);
            mix<N>(m2, arow, sl.T1);                           // M1[:,c] = (E A')[:,c]
            float m1[N];
            unpack_row<N>(m1, m2);
            __syncwarp();                                      // every lane has read the rows of D and E
            store_col<N>(sl.T0, c, m1);                        // rows of M1
        }
        __syncwarp();
        {
            f32x2 r2[N / 2];
            float cr[N];
            load_row<N>(cr, sl.C + c * LD);
            pack_row<N>(r2, cr);
            mix<N>(r2, arow, sl.T0);                           // row c of C2 = C + A M1
            unpack_row<N>(c2row, r2);
        }
        // symmetrise C2 and J2 through shared memory (row c against column c)
        store_row<N>(sl.T1 + c * LD, c2row);
        store_row<N>(sl.T2 + c * LD, j2);
        __syncwarp();
        float dmax = 0.f;
#pragma unroll
        for (int l = 0; l < N; ++l) {
            c2row[l] = 0.5f * (c2row[l] + sl.T1[l * LD + c]);
            j2[l] = 0.5f * (j2[l] + sl.T2[l * LD + c]);
            if (l == c)
                dmax = c2row[l];
        }
#pragma unroll
        for (int o = N / 2; o > 0; o >>= 1)
            dmax = fmaxf(dmax, __shfl_xor_sync(0xffffffffu, dmax, o, N));
        float g2[N];
#pragma unroll
        for (int l = 0; l < N; ++l)
            g2[l] = c2row[l];
        seg_chol_psd<N>(g2, c, 1e-7f * dmax);                  // row c of G2, C2 = G2 G2'
        if (active) {
            float4* dst = reinterpret_cast<float4*>(E + c * N);
#pragma unroll
            for (int l4 = 0; l4 < N / 4; ++l4) {
                dst[l4] = make_float4(a2row[4 * l4], a2row[4 * l4 + 1], a2row[4 * l4 + 2], a2row[4 * l4 + 3]);
                dst[N * N / 4 + l4] = make_float4(c2row[4 * l4], c2row[4 * l4 + 1], c2row[4 * l4 + 2], c2row[4 * l4 + 3]);
                dst[2 * N * N / 4 + l4] = make_float4(g2[4 * l4], g2[4 * l4 + 1], g2[4 * l4 + 2], g2[4 * l4 + 3]);
                dst[3 * N * N / 4 + l4] = make_float4(j2[4 * l4], j2[4 * l4 + 1], j2[4 * l4 + 2], j2[4 * l4 + 3]);
            }
        }
    }
}

// ---- forward loop of Alg. 1 from stored gains, status and NaN fill ------------------------------------------------------
template <int N>
struct RollSlot {
    float x[N], u[N];
};
template <int N>
__global__ void __launch_bounds__(THREADS) scan_rollout_kernel(ScanParams q)
{
    using S = Shape<N>;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const SolveParams& p = q.sp;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, sub = lane / N, c = lane % N;
    RollSlot<N>& sl = reinterpret_cast<RollSlot<N>*>(smem_raw)[warp * S::IPW + sub];
    const long long nwin = p.b0 * p.b1 * p.tcount;
    const int H = p.H;
    const float* Kall = p.K ? p.K : p.Kws;
    for (long long base = (long long)blockIdx.x * S::SLOTS; base < nwin; base += (long long)gridDim.x * S::SLOTS) {
        const long long w = base + warp * S::IPW + sub;
        const bool active = w < nwin;
        const long long inst = window_instance(p, active ? w : base);
        const int fail = q.fail_flag[inst];
        if (fail && active) {                                  // a failed instance only loses its outputs
            const float qn = quiet_nan();
            if (p.K)
                for (long long e = c; e < (long long)H * N * N; e += N)
                    p.K[inst * (long long)H * N * N + e] = qn;
            if (p.P) {
                const long long cnt = (long long)(p.first_only ? 1 : H + 1) * N * N;
                for (long long e = c; e < cnt; e += N)
                    p.P[inst * cnt + e] = qn;
            }
            if (p.x)
                for (long long e = c; e < (long long)(H + 1) * N; e += N)
                    p.x[inst * (long long)(H + 1) * N + e] = qn;
            if (p.u) {
                const long long cnt = p.first_only ? N : (long long)H * N;
                for (long long e = c; e < cnt; e += N)
                    p.u[inst * cnt + e] = qn;
            }
        }
        if (p.info && active && c == 0)
            p.info[inst] = fail;
        const bool ok = active && !fail;
        if (p.P && p.first_only && ok) {                       // P_0 out of the full buffer
            const float* src = q.Pbuf + inst * (long long)(H + 1) * N * N;
            float* dst = p.P + inst * (long long)N * N;
#pragma unroll 4
            for (int l = 0; l < N; ++l)
                dst[l * N + c] = src[l * N + c];
        }
        if (!(p.x || p.u))
            continue;
        const float* Ag = reinterpret_cast<const float*>(p.A.ptr) + operand_offset(p.A, inst, p.b1, p.b2);
        const float* Bg = reinterpret_cast<const float*>(p.B.ptr) + operand_offset(p.B, inst, p.b1, p.b2);
        float arow[N], brow[N];
#pragma unroll
        for (int l = 0; l < N; ++l) {
            arow[l] = __ldg(Ag + c * N + l);
            brow[l] = __ldg(Bg + c * N + l);
        }
        float* xo = (p.x && ok) ? p.x + inst * (long long)(H + 1) * N : nullptr;
        float* uo = (p.u && ok) ? p.u + inst * (long long)(p.first_only ? N : H * N) : nullptr;
        __syncwarp();
        sl.x[c] = load_elem(p.x0, operand_offset(p.x0, inst, p.b1, p.b2) + c);
        if (xo)
            xo[c] = sl.x[c];
        __syncwarp();
        const int steps = (p.x || !p.first_only) ? H : 1;
#pragma unroll 1
        for (int ts = 0; ts < steps; ++ts) {
            float xv[N];
            load_row<N>(xv, sl.x);
            const float4* kr = reinterpret_cast<const float4*>(Kall + (inst * (long long)H + ts) * N * N + c * N);
            float uc = 0.f;
#pragma unroll
            for (int l4 = 0; l4 < N / 4; ++l4) {
                const float4 k4 = kr[l4];
                uc = fmaf(k4.x, xv[4 * l4], uc);
                uc = fmaf(k4.y, xv[4 * l4 + 1], uc);
                uc = fmaf(k4.z, xv[4 * l4 + 2], uc);
                uc = fmaf(k4.w, xv[4 * l4 + 3], uc);
            }
            sl.u[c] = uc;
            if (uo && (!p.first_only || ts == 0))
                uo[(p.first_only ? 0 : ts * N) + c] = uc;
            __syncwarp();
            float uv[N];
            load_row<N>(uv, sl.u);
            float xc = 0.f;
#pragma unroll
            for (int l = 0; l < N; ++l)
                xc = fmaf(arow[l], xv[l], fmaf(brow[l], uv[l], xc));
            __syncwarp();                                      // x_t consumed by every lane
            sl.x[c] = xc;
            if (xo)
                xo[(long long)(ts + 1) * N + c] = xc;
            __syncwarp();
        }
    }
}

// Enqueue the whole scan for n = m = N: element of one step, log2(H) rounds of (applications, squaring), all gains,
// rollout.  Pbuf holds every P_t; elem is [N][4][n][n]; fail_flag is [N].
template <int N>
inline cudaError_t launch_scan_warp(const SolveParams& p, float* Pbuf, float* elem, int* fail_flag, int sm_count,
                                    cudaStream_t st, int* launches)
{
    using S = Shape<N>;
    cudaError_t e;
    ScanParams q;
    q.sp = p;
    q.elem = elem;
    q.Pbuf = Pbuf;
    q.fail_flag = fail_flag;
    q.step = 1;
    q.cnt = 1;
    q.gain_steps = 1;
    const long long nwin = p.b0 * p.b1 * p.tcount;
    const int H = p.H;
    int count = 0;
    auto blocks = [&](long long items, int per_sm) {
        long long g = (items + S::SLOTS - 1) / S::SLOTS;
        const long long cap = (long long)sm_count * per_sm * 4;
        return (unsigned)(g < 1 ? 1 : (g > cap ? cap : g));
    };
    const size_t sm_init = sizeof(InitSlot<N>) * S::SLOTS, sm_step = sizeof(StepSlot<N>) * S::SLOTS,
                 sm_sq = sizeof(SquareSlot<N>) * S::SLOTS, sm_roll = sizeof(RollSlot<N>) * S::SLOTS;
    if ((e = cudaFuncSetAttribute(scan_init_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_init))) return e;
    if ((e = cudaFuncSetAttribute(scan_step_kernel<N, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_step))) return e;
    if ((e = cudaFuncSetAttribute(scan_step_kernel<N, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_step))) return e;
    if ((e = cudaFuncSetAttribute(scan_square_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_sq))) return e;
    if ((e = cudaMemsetAsync(fail_flag, 0, sizeof(int) * (size_t)p.N, st))) return e;
    scan_init_kernel<N><<<blocks(nwin, 2), THREADS, sm_init, st>>>(q);
    if ((e = cudaGetLastError())) return e;
    ++count;
    for (int step = 1; step <= H; step <<= 1) {
        const int kend = (2 * step - 1 < H) ? 2 * step - 1 : H;
        q.step = step;
        q.cnt = kend - step + 1;
        scan_step_kernel<N, false><<<blocks(nwin * q.cnt, 2), THREADS, sm_step, st>>>(q);
        if ((e = cudaGetLastError())) return e;
        ++count;
        if (2 * step <= H) {
            scan_square_kernel<N><<<blocks(nwin, 1), THREADS, sm_sq, st>>>(q);
            if ((e = cudaGetLastError())) return e;
            ++count;
        }
    }
    const bool gains = p.K || p.x || p.u;
    q.gain_steps = (p.K || p.x || (p.u && !p.first_only)) ? H : 1;
    if (gains) {
        scan_step_kernel<N, true><<<blocks(nwin * q.gain_steps, 2), THREADS, sm_step, st>>>(q);
        if ((e = cudaGetLastError())) return e;
        ++count;
    }
    scan_rollout_kernel<N><<<blocks(nwin, 4), THREADS, sm_roll, st>>>(q);
    if ((e = cudaGetLastError())) return e;
    ++count;
    *launches = count;
    return cudaSuccess;
}

} // namespace scanw
} // namespace ttc
