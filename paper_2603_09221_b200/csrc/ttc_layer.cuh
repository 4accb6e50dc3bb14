// One Test-Time Control layer evaluation per (token, head): the LQR parameters are synthesised
// inside the kernel from the coefficient vectors (Contextualization / Parameterization paragraphs of
// the TTC-Net section) and the backward Riccati recursion (Prop. A.1 / Alg. 1) runs on them; nothing
// time-dependent is ever written to HBM.  Paper indices t = 1..T:
//     A_t = I + diag(exp(-t g_A) a)                 (diagonal)
//     B_t = Bbar diag(exp(-t g_B)),                 Bbar = sum_i s_B[i] B^(i)
//     Q_t = diag(exp(-t g_Q)) Qbar diag(exp(-t g_Q)),  Qbar = sum_i s_Q[i] Q^(i),  Q_0 = 0,
//     Q_T = sum_i s_Qf[i] Q^(i)                     (terminal override)
//     R_t = diag(1 / r_inv)
// and the layer output is the first optimal control u_1* = K_1 h_0.
//
// Same mapping as the dense fp32 warp kernel: N lanes own one instance, lane c holds COLUMN c of every
// symmetric matrix (= row c), cross-lane traffic goes through broadcast reads of the instance's rows in
// shared memory.  Step s = t - 1 (s = T-1 .. 0), P = P_{s+1}, with a = diag(A_t), g = exp(-t g_B), q = exp(-s g_Q):
//     V[:,c] = g_c (P Bbar[:,c])                     one dense contraction (rows of P broadcast)
//     T[:,c] = a_c P[:,c]                            A_t diagonal: no contraction
//     S[:,c] = e_c / r_inv_c + g .* (Bbar' V[:,c])   one pass over the rows of Bbar yields S and Y
//     Y[:,c] = g .* (Bbar' T[:,c])
//     Pn[:,c] = q_c (q .* Qbar[:,c]) [s >= 1] + a .* T[:,c]
//     S = L L',  Z[:,c] = L^{-1} Y[:,c],  Pn[:,c] -= Z' Z[:,c]        (P_s = Q_s + A'PA - Y'S^{-1}Y)
// and at s = 0 the gain column K[:,c] = -L^{-T} Z[:,c] for u_1* = K h_0.
// ttc_layer_kernel<N> is this one-column-per-lane form (used for N = 32); ttc_layer_kernel_c2<N> holds two columns
// per lane (used for N = 16), which halves the row reads per FMA.
#pragma once

#include "riccati_warp.cuh"

namespace ttc {
namespace layer {

struct LayerParams {
    long long N;                 // instances
    int T, r;
    const float *s_a, *s_ga, *s_gb, *s_gq;   // [N][n]
    const float *s_b, *s_q, *s_qf;           // [N][r]
    const float *r_inv, *h0;                 // [N][n]
    const float *B_basis, *Q_basis;          // [r][n][n]
    float* u1;                   // [N][n] or null
    float* P0;                   // [N][n][n] or null
    int* info;                   // [N] or null
    // gradient path only (ttc_layer_kernel<N, true>): every gain and the dual problem's first control are kept
    float* Kws;                  // [N][T][n][n]: K of step s = t - 1
    float* Pws;                  // [N][T][n][n]: P_s for 1 <= s <= T - 1 (slot 0 unused): the co-states are P_s x_s
    const float* g;              // [N][n]: dl/du_1*
    float* k0;                   // [N][n]: -S_0^{-1} g
};

using rwarp::Shape;
using rwarp::THREADS;
using rwarp::WARPS;

template <int N>
struct Smem {
    struct Slot {
        float buf0[Shape<N>::MAT];     // rows of P, then rows of Z
        float L[Shape<N>::MAT];        // staged V, then rows of L
        float Lt[Shape<N>::MAT];       // staged T, then rows of L'; K_1 rows at the last step
        float Bb[Shape<N>::MAT];       // rows of Bbar
        float rinv[N];                 // 1 / L[i][i]
        float x[N];                    // h_0
        float at[N], gb[N], gq[N];     // diag(A_t), exp(-t g_B), exp(-s g_Q) of the current step
    } slot[Shape<N>::SLOTS];
    int chunk;
};

// GRAD = the backward pass of the gradient entry point: the gain of EVERY step goes to p.Kws and, at the last step,
// k_0 = -S_0^{-1} g (the first control of the dual problem of Thm 3.2) to p.k0.
template <int N, bool GRAD = false>
__global__ void __launch_bounds__(THREADS, (N == 32) ? 3 : 4) ttc_layer_kernel(LayerParams p, int* chunk_counter)
{
    using S = Shape<N>;
    using namespace rwarp;
    constexpr int LD = S::LD;
    // n = 32: the dense contractions run on the tensor cores (three-pass tf32 mma.sync, see riccati_warp.cuh).  With a
    // diagonal A_t only three are left: V0 = P Bbar, Bbar'V0 and Z'Z; Y = G Bbar'P A_t is V0' scaled on both sides.
    constexpr bool MMA = (N == 32);
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem<N>& sm = *reinterpret_cast<Smem<N>*>(smem_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sub = lane / N, c = lane % N;
    typename Smem<N>::Slot& sl = sm.slot[warp * S::IPW + sub];
    const int T = p.T, r = p.r;
    const long long nchunks = (p.N + S::SLOTS - 1) / S::SLOTS;

    for (;;) {
        __syncthreads();
        if (tid == 0)
            sm.chunk = atomicAdd(chunk_counter, 1);
        __syncthreads();
        const long long chunk = sm.chunk;
        if (chunk >= nchunks)
            break;
        const long long inst_raw = chunk * S::SLOTS + warp * S::IPW + sub;
        const bool active = inst_raw < p.N;                   // idle segments shadow the chunk's first instance
        const long long inst = active ? inst_raw : chunk * S::SLOTS;

        // ---- synthesis of Bbar (rows -> shared), Qbar[:,c] (registers) and P_T = Q_T[:,c]
        float qcol[N], pcol[N];
        {
            float bcol[N];
#pragma unroll
            for (int l = 0; l < N; ++l) {
                bcol[l] = 0.f;
                qcol[l] = 0.f;
                pcol[l] = 0.f;
            }
            const float* sb = p.s_b + inst * r;
            const float* sq = p.s_q + inst * r;
            const float* sf = p.s_qf + inst * r;
#pragma unroll 1
            for (int i = 0; i < r; ++i) {
                const float wb = __ldg(sb + i), wq = __ldg(sq + i), wf = __ldg(sf + i);
                const float* Bi = p.B_basis + (long long)i * N * N + c;
                const float* Qi = p.Q_basis + (long long)i * N * N + c;
#pragma unroll
                for (int l = 0; l < N; ++l) {
                    const float qv = __ldg(Qi + l * N);
                    bcol[l] = fmaf(wb, __ldg(Bi + l * N), bcol[l]);
                    qcol[l] = fmaf(wq, qv, qcol[l]);
                    pcol[l] = fmaf(wf, qv, pcol[l]);
                }
            }
#pragma unroll
            for (int l = 0; l < N; ++l)
                sl.Bb[l * LD + c] = bcol[l];
        }
        const float a_c = __ldg(p.s_a + inst * N + c), ga_c = __ldg(p.s_ga + inst * N + c);
        const float gb_c = __ldg(p.s_gb + inst * N + c), gq_c = __ldg(p.s_gq + inst * N + c);
        const float r_c = 1.f / __ldg(p.r_inv + inst * N + c);
        sl.x[c] = __ldg(p.h0 + inst * N + c);
        store_row<N>(sl.buf0 + c * LD, pcol);                 // rows of P_T (row c = column c)
        int fail = 0;

#pragma unroll 1
        for (int s = T - 1; s >= 0; --s) {
            const float tt = (float)(s + 1);
            const float at_c = fmaf(__expf(-tt * ga_c), a_c, 1.f);
            const float g_c = __expf(-tt * gb_c);
            const float q_c = (s >= 1) ? __expf(-(float)s * gq_c) : 0.f;     // Q_0 = 0
            sl.at[c] = at_c;
            sl.gb[c] = g_c;
            sl.gq[c] = q_c;
            __syncwarp();                                     // rows of P and the step's diagonals are in place
            float sv[N], y[N], pn[N];
            // Tensor-core path: one copy of the product code run in three phases (V0 = P Bbar -> rows of L, Bbar'V0 ->
            // rows of L', then factorisation / substitutions / gains and Z'Z -> rows of L).  Otherwise only phase 2.
#pragma unroll 1
            for (int ph = MMA ? 0 : 2; ph < 3; ++ph) {
            if (!MMA || ph == 2) {
            if constexpr (MMA) {
                float gv[N], av[N], qv[N], v0[N];
                load_row<N>(gv, sl.gb);
                load_row<N>(av, sl.at);
                load_row<N>(qv, sl.gq);
                load_row<N>(v0, sl.L + c * LD);               // row c of V0 = column c of Bbar'P
#pragma unroll
                for (int l = 0; l < N; ++l) {
                    sv[l] = gv[l] * g_c * sl.Lt[l * LD + c];  // S = G Bbar'P Bbar G + R
                    y[l] = gv[l] * at_c * v0[l];              // Y = G Bbar'P A_t
                    pn[l] = fmaf(q_c * qv[l], qcol[l], av[l] * at_c * pcol[l]);
                    if (l == c)
                        sv[l] += r_c;
                }
            } else {
                f32x2 vcol[N / 2];
#pragma unroll
                for (int k = 0; k < N / 2; ++k)
                    vcol[k] = 0ull;
#pragma unroll 4
                for (int i = 0; i < N; ++i) {                     // P Bbar[:,c]
                    const float bic = sl.Bb[i * LD + c];
                    axpy_row<N>(vcol, bic, sl.buf0 + i * LD);
                }
                // stage V[:,c] = g_c (P Bbar[:,c]) so that the next loop can run over k without indexing registers
                // dynamically.  With a diagonal A_t, Y = G Bbar'P A_t is the transpose of V scaled by a_c: column c of Y
                // is row c of the staged matrix, and the contraction Bbar'T is not needed.
#pragma unroll
                for (int k = 0; k < N / 2; ++k) {
                    float v0, v1;
                    unpack2(vcol[k], v0, v1);
                    sl.L[(2 * k) * LD + c] = g_c * v0;
                    sl.L[(2 * k + 1) * LD + c] = g_c * v1;
                }
                __syncwarp();
                f32x2 s2[N / 2];
#pragma unroll
                for (int l = 0; l < N / 2; ++l)
                    s2[l] = 0ull;
#pragma unroll 4
                for (int k = 0; k < N; ++k)                       // Bbar' V[:,c]
                    axpy_row<N>(s2, sl.L[k * LD + c], sl.Bb + k * LD);
                unpack_row<N>(sv, s2);
                load_row<N>(y, sl.L + c * LD);                    // g_l (Bbar'P)[l][c]
                {
                    float gv[N], av[N], qv[N];
                    load_row<N>(gv, sl.gb);
                    load_row<N>(av, sl.at);
                    load_row<N>(qv, sl.gq);
#pragma unroll
                    for (int l = 0; l < N; ++l) {
                        sv[l] *= gv[l];
                        y[l] *= at_c;
                        // Pn[l][c] = q_l Qbar[l][c] q_c + a_l a_c P[l][c]
                        pn[l] = fmaf(q_c * qv[l], qcol[l], av[l] * at_c * pcol[l]);
                        if (l == c)
                            sv[l] += r_c;
                    }
                }
            }
            float rs_own;
            const int bad = seg_chol<N>(sv, rs_own, c);
            if (bad && !fail)
                fail = s * N + bad;
            __syncwarp();                                     // every lane is done with the rows of P in buf0 and the staged columns
            store_row<N>(sl.L + c * LD, sv);
#pragma unroll
            for (int k = 0; k < N; ++k)
                sl.Lt[k * LD + c] = sv[k];
            sl.rinv[c] = rs_own;
            __syncwarp();
            float rinv[N];
            load_row<N>(rinv, sl.rinv);
#pragma unroll
            for (int k = 0; k < N; ++k) {                     // Z[:,c] = L^{-1} Y[:,c]
                const float zk = y[k] * rinv[k];
                y[k] = zk;
                const float* lt = sl.Lt + k * LD;
#pragma unroll
                for (int i4 = (k + 1) & ~3; i4 < N; i4 += 4) {
                    const float4 l4 = *reinterpret_cast<const float4*>(lt + i4);
                    if (i4 + 0 > k) y[i4 + 0] = fmaf(-l4.x, zk, y[i4 + 0]);
                    if (i4 + 1 > k) y[i4 + 1] = fmaf(-l4.y, zk, y[i4 + 1]);
                    if (i4 + 2 > k) y[i4 + 2] = fmaf(-l4.z, zk, y[i4 + 2]);
                    if (i4 + 3 > k) y[i4 + 3] = fmaf(-l4.w, zk, y[i4 + 3]);
                }
            }
#pragma unroll
            for (int q = 0; q < N; ++q)
                sl.buf0[q * LD + c] = y[q];                   // rows of Z
            __syncwarp();
            if constexpr (!MMA) {
                f32x2 p2[N / 2];
                pack_row<N>(p2, pn);
#pragma unroll 4
                for (int q = 0; q < N; ++q)                   // Pn[:,c] -= Z' Z[:,c]
                    axpy_row<N>(p2, -sl.buf0[q * LD + c], sl.buf0 + q * LD);
                unpack_row<N>(pcol, p2);
            }
            if (GRAD || (s == 0 && p.u1)) {                   // K[:,c] = -L^{-T} Z[:,c]; rows of K -> Lt
#pragma unroll
                for (int k = N - 1; k >= 0; --k) {
                    const float xk = y[k] * rinv[k];
                    y[k] = xk;
                    const float* lr = sl.L + k * LD;
#pragma unroll
                    for (int i4 = 0; i4 < k; i4 += 4) {
                        const float4 l4 = *reinterpret_cast<const float4*>(lr + i4);
                        if (i4 + 0 < k) y[i4 + 0] = fmaf(-l4.x, xk, y[i4 + 0]);
                        if (i4 + 1 < k) y[i4 + 1] = fmaf(-l4.y, xk, y[i4 + 1]);
                        if (i4 + 2 < k) y[i4 + 2] = fmaf(-l4.z, xk, y[i4 + 2]);
                        if (i4 + 3 < k) y[i4 + 3] = fmaf(-l4.w, xk, y[i4 + 3]);
                    }
                }
                if (GRAD) {
                    if (active) {
                        float* kt = p.Kws + (inst * (long long)T + s) * N * N + c;
#pragma unroll
                        for (int l = 0; l < N; ++l)
                            kt[l * N] = -y[l];
                    }
                    if (s == 0) {
                        // k_0 = -L^{-T} L^{-1} g with one component per lane: the pivot's value travels by shuffle,
                        // lane i reads its own rows of L and L'
                        float gz = __ldg(p.g + inst * N + c);
                        const float rown = sl.rinv[c];
#pragma unroll 4
                        for (int k = 0; k < N; ++k) {
                            const float zk = __shfl_sync(0xffffffffu, gz * rown, k, N);
                            if (c > k)
                                gz = fmaf(-sl.L[c * LD + k], zk, gz);
                            else if (c == k)
                                gz = zk;
                        }
#pragma unroll 4
                        for (int k = N - 1; k >= 0; --k) {
                            const float xk = __shfl_sync(0xffffffffu, gz * rown, k, N);
                            if (c < k)
                                gz = fmaf(-sl.Lt[c * LD + k], xk, gz);
                            else if (c == k)
                                gz = xk;
                        }
                        if (active)
                            p.k0[inst * N + c] = -gz;
                    }
                }
                if (s == 0) {
                    if (GRAD)
                        __syncwarp();                         // every lane is done with L' (the substitution of g)
#pragma unroll
                    for (int l = 0; l < N; ++l)
                        sl.Lt[l * LD + c] = -y[l];
                }
            }
            }                                                 // phase 2: factorisation, substitutions, gains
            if constexpr (MMA) {
                // phase:  0       1        2
                // A'   :  P       Bbar'    Z'
                // B    :  Bbar    V0       Z
                // to   :  L       L'       L     (the rows of L' may hold K_1 by then)
                const float* Am = ph == 1 ? sl.Bb : sl.buf0;
                const float* Bm = ph == 0 ? sl.Bb : ph == 1 ? sl.L : sl.buf0;
                float* Dm = ph == 1 ? sl.Lt : sl.L;
                __syncwarp();                                 // every lane is done with what the operands replace
                float acc[2][4][4];
                mma32_zero(acc);
                mma32_product(acc, Am, Bm, lane);
                __syncwarp();
                mma32_store(Dm, acc, lane);
                __syncwarp();
                if (ph == 2) {
                    // P_s[:,c] = Pn[:,c] - Z'Z[:,c], with Z'Z averaged with its transpose: Pn is symmetric bit for bit
                    // (the FP32 loops keep Z'Z so too), the three-pass product is only up to rounding, and an
                    // antisymmetric part E obeys E <- A_t E A_t, which grows wherever the diagonal of A_t exceeds one
                    float zr[N];
                    load_row<N>(zr, sl.L + c * LD);
#pragma unroll
                    for (int l = 0; l < N; ++l)
                        pcol[l] = pn[l] - 0.5f * (sl.L[l * LD + c] + zr[l]);
                }
            }
            }                                                 // phases
            __syncwarp();                                     // rows of Z consumed
            store_row<N>(sl.buf0 + c * LD, pcol);             // rows of P_s (row c = column c)
            if (GRAD && s >= 1 && active) {
                float* pt = p.Pws + (inst * (long long)T + s) * N * N + c;
#pragma unroll
                for (int l = 0; l < N; ++l)
                    pt[l * N] = pcol[l];
            }
        }
        __syncwarp();

        const bool store_ok = active && !fail;
        if (p.P0 && active) {
            float* pt = p.P0 + inst * (long long)N * N + c;
            const float qn = quiet_nan();
#pragma unroll
            for (int l = 0; l < N; ++l)
                pt[l * N] = fail ? qn : pcol[l];
        }
        if (p.u1) {                                           // u_1* = K_1 h_0: lane c takes row c of K_1
            float kr[N], xv[N];
            load_row<N>(kr, sl.Lt + c * LD);
            load_row<N>(xv, sl.x);
            float uc = 0.f;
#pragma unroll
            for (int j = 0; j < N; ++j)
                uc = fmaf(kr[j], xv[j], uc);
            if (active)
                p.u1[inst * (long long)N + c] = store_ok ? uc : quiet_nan();
        }
        if (p.info && active && c == 0)
            p.info[inst] = fail;
    }
}

// ---- two columns per lane ---------------------------------------------------------------------------------------
// Same computation with N / 2 lanes per instance: lane j holds columns 2j and 2j + 1 of every matrix, so that one
// broadcast read of a matrix row feeds the packed FMAs of two columns (the one-column kernel is bound by the
// shared-memory pipe).  Four instances per warp when N = 16.
template <int N>
struct Shape2 {
    static constexpr int LD = N + 4;
    static constexpr int G = N / 2;                 // lanes per instance
    static constexpr int IPW = 32 / G;
    static constexpr int SLOTS = WARPS * IPW;
    static constexpr int MAT = N * LD;
};
template <int N>
struct Smem2 {
    struct Slot {
        float buf0[Shape2<N>::MAT], L[Shape2<N>::MAT], Lt[Shape2<N>::MAT], Bb[Shape2<N>::MAT];
        float rinv[N], x[N], at[N], gb[N], gq[N];
    } slot[Shape2<N>::SLOTS];
    int chunk;
};

// Cholesky of an N x N SPD matrix spread over N / 2 lanes: lane j holds rows 2j (s0) and 2j + 1 (s1) (= columns, by
// symmetry).  On return s0, s1 hold the rows of L (entries right of the diagonal are meaningless), rs0 / rs1 the
// reciprocals of their diagonal entries.  Returns 0 or 1 + the index of the first non-positive pivot.
template <int N>
__device__ __forceinline__ int seg_chol2(float (&s0)[N], float (&s1)[N], float& rs0, float& rs1, int j)
{
    constexpr int G = N / 2;
    int bad = 0;
    rs0 = rs1 = 1.f;
#pragma unroll
    for (int p = 0; p < N; ++p) {
        const float a0 = s0[p], a1 = s1[p];
        float d = __shfl_sync(0xffffffffu, (p & 1) ? a1 : a0, p >> 1, G);
        if (!(d > 0.f)) {
            if (!bad)
                bad = p + 1;
            d = 1.f;
        }
        const float rinv = __frcp_rn(d);
        const float f0 = a0 * rinv, f1 = a1 * rinv;
#pragma unroll
        for (int cc = p + 1; cc < N; ++cc) {
            const float lc = __shfl_sync(0xffffffffu, (cc & 1) ? a1 : a0, cc >> 1, G);
            s0[cc] = fmaf(-f0, lc, s0[cc]);
            s1[cc] = fmaf(-f1, lc, s1[cc]);
        }
        const float rs = rsqrtf(d);
        s0[p] = a0 * rs;
        s1[p] = a1 * rs;
        if (2 * j == p)
            rs0 = rs;
        if (2 * j + 1 == p)
            rs1 = rs;
    }
    return bad;
}

// acc0[l] += w0 * row[l], acc1[l] += w1 * row[l]: one pass over the row for two columns
template <int N>
__device__ __forceinline__ void axpy_row2(rwarp::f32x2 (&acc0)[N / 2], rwarp::f32x2 (&acc1)[N / 2], float w0, float w1, const float* row)
{
    const rwarp::f32x2 ww0 = rwarp::pack2(w0, w0), ww1 = rwarp::pack2(w1, w1);
#pragma unroll
    for (int q = 0; q < N / 4; ++q) {
        const ulonglong2 t = *reinterpret_cast<const ulonglong2*>(row + 4 * q);
        rwarp::fma2(acc0[2 * q], ww0, t.x);
        rwarp::fma2(acc0[2 * q + 1], ww0, t.y);
        rwarp::fma2(acc1[2 * q], ww1, t.x);
        rwarp::fma2(acc1[2 * q + 1], ww1, t.y);
    }
}

// GRAD: as in ttc_layer_kernel (every K_s, every P_s with s >= 1 and k_0 = -S_0^{-1} g are kept).
template <int N, bool GRAD = false>
__global__ void __launch_bounds__(THREADS, 2) ttc_layer_kernel_c2(LayerParams p, int* chunk_counter)
{
    using S = Shape2<N>;
    using namespace rwarp;
    constexpr int LD = S::LD, G = S::G;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem2<N>& sm = *reinterpret_cast<Smem2<N>*>(smem_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sub = lane / G, j = lane % G;
    const int c0 = 2 * j, c1 = 2 * j + 1;
    typename Smem2<N>::Slot& sl = sm.slot[warp * S::IPW + sub];
    const int T = p.T, r = p.r;
    const long long nchunks = (p.N + S::SLOTS - 1) / S::SLOTS;

    for (;;) {
        __syncthreads();
        if (tid == 0)
            sm.chunk = atomicAdd(chunk_counter, 1);
        __syncthreads();
        const long long chunk = sm.chunk;
        if (chunk >= nchunks)
            break;
        const long long inst_raw = chunk * S::SLOTS + warp * S::IPW + sub;
        const bool active = inst_raw < p.N;                   // idle segments shadow the chunk's first instance
        const long long inst = active ? inst_raw : chunk * S::SLOTS;

        // ---- synthesis of Bbar (rows -> shared), Qbar[:, c0..c1] (registers) and P_T = Q_T[:, c0..c1]
        float q0[N], q1[N], p0[N], p1[N];
        {
            float b0[N], b1[N];
#pragma unroll
            for (int l = 0; l < N; ++l)
                b0[l] = b1[l] = q0[l] = q1[l] = p0[l] = p1[l] = 0.f;
            const float* sb = p.s_b + inst * r;
            const float* sq = p.s_q + inst * r;
            const float* sf = p.s_qf + inst * r;
#pragma unroll 1
            for (int i = 0; i < r; ++i) {
                const float wb = __ldg(sb + i), wq = __ldg(sq + i), wf = __ldg(sf + i);
                const float2* Bi = reinterpret_cast<const float2*>(p.B_basis + (long long)i * N * N + c0);
                const float2* Qi = reinterpret_cast<const float2*>(p.Q_basis + (long long)i * N * N + c0);
#pragma unroll
                for (int l = 0; l < N; ++l) {
                    const float2 bv = __ldg(Bi + l * (N / 2)), qv = __ldg(Qi + l * (N / 2));
                    b0[l] = fmaf(wb, bv.x, b0[l]);
                    b1[l] = fmaf(wb, bv.y, b1[l]);
                    q0[l] = fmaf(wq, qv.x, q0[l]);
                    q1[l] = fmaf(wq, qv.y, q1[l]);
                    p0[l] = fmaf(wf, qv.x, p0[l]);
                    p1[l] = fmaf(wf, qv.y, p1[l]);
                }
            }
#pragma unroll
            for (int l = 0; l < N; ++l)
                *reinterpret_cast<float2*>(sl.Bb + l * LD + c0) = make_float2(b0[l], b1[l]);
        }
        const float2 a_c = __ldg(reinterpret_cast<const float2*>(p.s_a + inst * N + c0));
        const float2 ga_c = __ldg(reinterpret_cast<const float2*>(p.s_ga + inst * N + c0));
        const float2 gb_c = __ldg(reinterpret_cast<const float2*>(p.s_gb + inst * N + c0));
        const float2 gq_c = __ldg(reinterpret_cast<const float2*>(p.s_gq + inst * N + c0));
        const float2 ri_c = __ldg(reinterpret_cast<const float2*>(p.r_inv + inst * N + c0));
        const float r_0 = 1.f / ri_c.x, r_1 = 1.f / ri_c.y;
        *reinterpret_cast<float2*>(sl.x + c0) = __ldg(reinterpret_cast<const float2*>(p.h0 + inst * N + c0));
        store_row<N>(sl.buf0 + c0 * LD, p0);                  // rows of P_T (row c = column c)
        store_row<N>(sl.buf0 + c1 * LD, p1);
        int fail = 0;

#pragma unroll 1
        for (int s = T - 1; s >= 0; --s) {
            const float tt = (float)(s + 1);
            const float at0 = fmaf(__expf(-tt * ga_c.x), a_c.x, 1.f), at1 = fmaf(__expf(-tt * ga_c.y), a_c.y, 1.f);
            const float g0 = __expf(-tt * gb_c.x), g1 = __expf(-tt * gb_c.y);
            const float qq0 = (s >= 1) ? __expf(-(float)s * gq_c.x) : 0.f;       // Q_0 = 0
            const float qq1 = (s >= 1) ? __expf(-(float)s * gq_c.y) : 0.f;
            *reinterpret_cast<float2*>(sl.at + c0) = make_float2(at0, at1);
            *reinterpret_cast<float2*>(sl.gb + c0) = make_float2(g0, g1);
            *reinterpret_cast<float2*>(sl.gq + c0) = make_float2(qq0, qq1);
            __syncwarp();                                     // rows of P and the step's diagonals are in place
            float v0[N], v1[N];
            {
                f32x2 a0[N / 2], a1[N / 2];
#pragma unroll
                for (int k = 0; k < N / 2; ++k)
                    a0[k] = a1[k] = 0ull;
#pragma unroll 4
                for (int i = 0; i < N; ++i) {                 // P Bbar[:, c0..c1]
                    const float2 b = *reinterpret_cast<const float2*>(sl.Bb + i * LD + c0);
                    axpy_row2<N>(a0, a1, b.x, b.y, sl.buf0 + i * LD);
                }
                unpack_row<N>(v0, a0);
                unpack_row<N>(v1, a1);
            }
            // V[:, c] = g_c (P Bbar)[:, c] goes to the rows of L (free until the factor is published): with a diagonal A_t,
            // Y = G Bbar'P A_t is the transpose of V scaled by a_c, so column c of Y is row c of that buffer and the
            // contraction Bbar'T is not needed
#pragma unroll
            for (int k = 0; k < N; ++k)
                *reinterpret_cast<float2*>(sl.L + k * LD + c0) = make_float2(g0 * v0[k], g1 * v1[k]);
            __syncwarp();
            f32x2 s20[N / 2], s21[N / 2];
#pragma unroll
            for (int l = 0; l < N / 2; ++l)
                s20[l] = s21[l] = 0ull;
            // fully unrolled: V[k][c] = g_c v[k] comes straight from registers
#pragma unroll
            for (int k = 0; k < N; ++k) {                     // Bbar' V for both columns: each row of Bbar read once
                const f32x2 w0 = pack2(g0 * v0[k], g0 * v0[k]), w1 = pack2(g1 * v1[k], g1 * v1[k]);
#pragma unroll
                for (int q = 0; q < N / 4; ++q) {
                    const ulonglong2 b4 = *reinterpret_cast<const ulonglong2*>(sl.Bb + k * LD + 4 * q);
                    fma2(s20[2 * q], w0, b4.x);
                    fma2(s20[2 * q + 1], w0, b4.y);
                    fma2(s21[2 * q], w1, b4.x);
                    fma2(s21[2 * q + 1], w1, b4.y);
                }
            }
            float s0[N], s1[N], y0[N], y1[N], pn0[N], pn1[N];
            unpack_row<N>(s0, s20);
            unpack_row<N>(s1, s21);
            load_row<N>(y0, sl.L + c0 * LD);                  // g_l (Bbar'P)[l][c0]
            load_row<N>(y1, sl.L + c1 * LD);
            {
                float gv[N], av[N], qv[N];
                load_row<N>(gv, sl.gb);
                load_row<N>(av, sl.at);
                load_row<N>(qv, sl.gq);
#pragma unroll
                for (int l = 0; l < N; ++l) {
                    s0[l] *= gv[l];
                    s1[l] *= gv[l];
                    y0[l] *= at0;
                    y1[l] *= at1;
                    pn0[l] = fmaf(qq0 * qv[l], q0[l], av[l] * at0 * p0[l]);
                    pn1[l] = fmaf(qq1 * qv[l], q1[l], av[l] * at1 * p1[l]);
                    if (l == c0)
                        s0[l] += r_0;
                    if (l == c1)
                        s1[l] += r_1;
                }
            }
            float rs0, rs1;
            const int bad = seg_chol2<N>(s0, s1, rs0, rs1, j);
            if (bad && !fail)
                fail = s * N + bad;
            __syncwarp();                                     // every lane is done with the rows of P in buf0
            store_row<N>(sl.L + c0 * LD, s0);
            store_row<N>(sl.L + c1 * LD, s1);
#pragma unroll
            for (int k = 0; k < N; ++k)
                *reinterpret_cast<float2*>(sl.Lt + k * LD + c0) = make_float2(s0[k], s1[k]);
            *reinterpret_cast<float2*>(sl.rinv + c0) = make_float2(rs0, rs1);
            __syncwarp();
            float rinv[N];
            load_row<N>(rinv, sl.rinv);
#pragma unroll
            for (int k = 0; k < N; ++k) {                     // Z[:, c] = L^{-1} Y[:, c] for both columns
                const float z0 = y0[k] * rinv[k], z1 = y1[k] * rinv[k];
                y0[k] = z0;
                y1[k] = z1;
                const float* lt = sl.Lt + k * LD;
#pragma unroll
                for (int i4 = (k + 1) & ~3; i4 < N; i4 += 4) {
                    const float4 l4 = *reinterpret_cast<const float4*>(lt + i4);
                    if (i4 + 0 > k) { y0[i4 + 0] = fmaf(-l4.x, z0, y0[i4 + 0]); y1[i4 + 0] = fmaf(-l4.x, z1, y1[i4 + 0]); }
                    if (i4 + 1 > k) { y0[i4 + 1] = fmaf(-l4.y, z0, y0[i4 + 1]); y1[i4 + 1] = fmaf(-l4.y, z1, y1[i4 + 1]); }
                    if (i4 + 2 > k) { y0[i4 + 2] = fmaf(-l4.z, z0, y0[i4 + 2]); y1[i4 + 2] = fmaf(-l4.z, z1, y1[i4 + 2]); }
                    if (i4 + 3 > k) { y0[i4 + 3] = fmaf(-l4.w, z0, y0[i4 + 3]); y1[i4 + 3] = fmaf(-l4.w, z1, y1[i4 + 3]); }
                }
            }
#pragma unroll
            for (int q = 0; q < N; ++q)
                *reinterpret_cast<float2*>(sl.buf0 + q * LD + c0) = make_float2(y0[q], y1[q]);     // rows of Z
            __syncwarp();
            {
                f32x2 p20[N / 2], p21[N / 2];
                pack_row<N>(p20, pn0);
                pack_row<N>(p21, pn1);
#pragma unroll
                for (int q = 0; q < N; ++q)                   // Pn[:, c] -= Z' Z[:, c]
                    axpy_row2<N>(p20, p21, -y0[q], -y1[q], sl.buf0 + q * LD);
                unpack_row<N>(p0, p20);
                unpack_row<N>(p1, p21);
            }
            if (GRAD || (s == 0 && p.u1)) {                   // K[:, c] = -L^{-T} Z[:, c]; rows of K -> Lt
#pragma unroll
                for (int k = N - 1; k >= 0; --k) {
                    const float x0 = y0[k] * rinv[k], x1 = y1[k] * rinv[k];
                    y0[k] = x0;
                    y1[k] = x1;
                    const float* lr = sl.L + k * LD;
#pragma unroll
                    for (int i4 = 0; i4 < k; i4 += 4) {
                        const float4 l4 = *reinterpret_cast<const float4*>(lr + i4);
                        if (i4 + 0 < k) { y0[i4 + 0] = fmaf(-l4.x, x0, y0[i4 + 0]); y1[i4 + 0] = fmaf(-l4.x, x1, y1[i4 + 0]); }
                        if (i4 + 1 < k) { y0[i4 + 1] = fmaf(-l4.y, x0, y0[i4 + 1]); y1[i4 + 1] = fmaf(-l4.y, x1, y1[i4 + 1]); }
                        if (i4 + 2 < k) { y0[i4 + 2] = fmaf(-l4.z, x0, y0[i4 + 2]); y1[i4 + 2] = fmaf(-l4.z, x1, y1[i4 + 2]); }
                        if (i4 + 3 < k) { y0[i4 + 3] = fmaf(-l4.w, x0, y0[i4 + 3]); y1[i4 + 3] = fmaf(-l4.w, x1, y1[i4 + 3]); }
                    }
                }
                if (GRAD) {
                    if (active) {
                        float* kt = p.Kws + (inst * (long long)T + s) * N * N + c0;
#pragma unroll
                        for (int l = 0; l < N; ++l)
                            *reinterpret_cast<float2*>(kt + l * N) = make_float2(-y0[l], -y1[l]);
                    }
                    if (s == 0) {
                        // k_0 = -L^{-T} L^{-1} g, two components per lane: the pivot's value travels by shuffle, a lane
                        // reads its own rows of L and L'
                        const float2 gg = __ldg(reinterpret_cast<const float2*>(p.g + inst * N + c0));
                        float gz0 = gg.x, gz1 = gg.y;
                        const float r0 = sl.rinv[c0], r1 = sl.rinv[c1];
#pragma unroll 4
                        for (int k = 0; k < N; ++k) {
                            const float zk = __shfl_sync(0xffffffffu, (k & 1) ? gz1 * r1 : gz0 * r0, k >> 1, G);
                            if (c0 > k) gz0 = fmaf(-sl.L[c0 * LD + k], zk, gz0); else if (c0 == k) gz0 = zk;
                            if (c1 > k) gz1 = fmaf(-sl.L[c1 * LD + k], zk, gz1); else if (c1 == k) gz1 = zk;
                        }
#pragma unroll 4
                        for (int k = N - 1; k >= 0; --k) {
                            const float xk = __shfl_sync(0xffffffffu, (k & 1) ? gz1 * r1 : gz0 * r0, k >> 1, G);
                            if (c0 < k) gz0 = fmaf(-sl.Lt[c0 * LD + k], xk, gz0); else if (c0 == k) gz0 = xk;
                            if (c1 < k) gz1 = fmaf(-sl.Lt[c1 * LD + k], xk, gz1); else if (c1 == k) gz1 = xk;
                        }
                        if (active)
                            *reinterpret_cast<float2*>(p.k0 + inst * N + c0) = make_float2(-gz0, -gz1);
                        __syncwarp();                         // every lane is done with L' (the substitution of g)
                    }
                }
                if (s == 0) {
#pragma unroll
                    for (int l = 0; l < N; ++l)
                        *reinterpret_cast<float2*>(sl.Lt + l * LD + c0) = make_float2(-y0[l], -y1[l]);
                }
            }
            __syncwarp();                                     // rows of Z consumed
            store_row<N>(sl.buf0 + c0 * LD, p0);              // rows of P_s (row c = column c)
            store_row<N>(sl.buf0 + c1 * LD, p1);
            if (GRAD && s >= 1 && active) {
                float* pt = p.Pws + (inst * (long long)T + s) * N * N + c0;
#pragma unroll
                for (int l = 0; l < N; ++l)
                    *reinterpret_cast<float2*>(pt + l * N) = make_float2(p0[l], p1[l]);
            }
        }
        __syncwarp();

        const bool store_ok = active && !fail;
        const float qn = quiet_nan();
        if (p.P0 && active) {
            float* pt = p.P0 + inst * (long long)N * N + c0;
#pragma unroll
            for (int l = 0; l < N; ++l)
                *reinterpret_cast<float2*>(pt + l * N) = fail ? make_float2(qn, qn) : make_float2(p0[l], p1[l]);
        }
        if (p.u1) {                                           // u_1* = K_1 h_0: lane j takes rows c0, c1 of K_1
            float k0[N], k1[N], xv[N];
            load_row<N>(k0, sl.Lt + c0 * LD);
            load_row<N>(k1, sl.Lt + c1 * LD);
            load_row<N>(xv, sl.x);
            float u0 = 0.f, u1v = 0.f;
#pragma unroll
            for (int l = 0; l < N; ++l) {
                u0 = fmaf(k0[l], xv[l], u0);
                u1v = fmaf(k1[l], xv[l], u1v);
            }
            if (active)
                *reinterpret_cast<float2*>(p.u1 + inst * (long long)N + c0) = store_ok ? make_float2(u0, u1v) : make_float2(qn, qn);
        }
        if (p.info && active && j == 0)
            p.info[inst] = fail;
    }
}

template <int N>
inline size_t smem_bytes_c2() { return sizeof(Smem2<N>); }

template <int N>
inline size_t smem_bytes() { return sizeof(Smem<N>); }

} // namespace layer
} // namespace ttc
