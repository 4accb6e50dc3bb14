// BASELINE, not the solver: the reverse symplectic iteration of Thm 3.3 with row normalisation (the fused kernel the
// paper describes in its hardware co-design appendix), restated for the contextualised layer's parameters so that it
// can be timed and checked beside ttc_layer_kernel on the same inputs.
//
//     [Y1 Y2] = [I  Q_T] Sigma_T ... Sigma_1,      Sigma_t = [I 0; G_t I] diag(A_t^{-T}, A_t) [I Q_{t-1}; 0 I],
//     G_t = B_t R_t^{-1} B_t',     P_0 = Y1^{-1} Y2,     lambda_0 = P_0 h_0,     u_1 = -R_1^{-1} B_1' A_1^{-T} lambda_0.
// Right-multiplying a row [y1 y2] by Sigma_t touches that row only, so lane i of an N-lane segment owns row i of
// [Y1 Y2] in registers; per step, with a = diag(A_t), g = exp(-t g_B), q = exp(-(t-1) g_Q) (q = 0 at t = 1: Q_0 = 0):
//     y3 = (y2 Bbar) .* g .* r_inv           y1 <- (y1 + (y3 .* g) Bbar') ./ a
//     y2 <- y2 .* a + ((y1 .* q) Qbar) .* q   then both rows are divided by max(|y1|_1, |y2|_1).
// Y1 P_0 = Y2 is solved by Gauss-Jordan elimination with partial pivoting across the lanes (shuffles).
// The product contains A_t^{-1} and is a shooting method: in float32 it loses the result within a few tens of
// steps on inputs where the backward recursion stays at rounding level (measured in the tests and the sweep).
#pragma once

#include "ttc_layer.cuh"
#include "scan_warp.cuh"

namespace ttc {
namespace sigma {

using rwarp::Shape;
using rwarp::THREADS;
using rwarp::f32x2;
using rwarp::pack_row;
using rwarp::unpack_row;
using scanw::mix;
using scanw::zero2;

template <int N>
struct Slot {
    float Bb[Shape<N>::MAT];       // rows of Bbar
    float Bt[Shape<N>::MAT];       // rows of Bbar'
    float Qb[Shape<N>::MAT];       // rows of Qbar
    float vec[N];                  // lambda_0 ./ a_1
    float sa[N], ga[N], gb[N], gq[N], ri[N];     // s_a, the three decay rates, diag(R^{-1})
};

template <int N>
__global__ void __launch_bounds__(THREADS, 1) sigma_product_kernel(layer::LayerParams p)
{
    using S = Shape<N>;
    constexpr int LD = S::LD;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, sub = lane / N, c = lane % N;
    Slot<N>& sl = reinterpret_cast<Slot<N>*>(smem_raw)[warp * S::IPW + sub];
    const int T = p.T, r = p.r;
    for (long long base = (long long)blockIdx.x * S::SLOTS; base < p.N; base += (long long)gridDim.x * S::SLOTS) {
        const long long raw = base + warp * S::IPW + sub;
        const bool active = raw < p.N;
        const long long inst = active ? raw : base;
        __syncwarp();
        // ---- synthesis: lane c forms column c of Bbar and Qbar, and row c of Q_T (symmetric) as the start of y2
        float y1[N], y2[N];
        {
            float bcol[N], qcol[N];
#pragma unroll
            for (int l = 0; l < N; ++l) {
                bcol[l] = 0.f;
                qcol[l] = 0.f;
                y2[l] = 0.f;
                y1[l] = (l == c) ? 1.f : 0.f;
            }
#pragma unroll 1
            for (int i = 0; i < r; ++i) {
                const float wb = __ldg(p.s_b + inst * r + i), wq = __ldg(p.s_q + inst * r + i), wf = __ldg(p.s_qf + inst * r + i);
                const float* Bi = p.B_basis + (long long)i * N * N + c;
                const float* Qi = p.Q_basis + (long long)i * N * N + c;
#pragma unroll
                for (int l = 0; l < N; ++l) {
                    const float qv = __ldg(Qi + l * N);
                    bcol[l] = fmaf(wb, __ldg(Bi + l * N), bcol[l]);
                    qcol[l] = fmaf(wq, qv, qcol[l]);
                    y2[l] = fmaf(wf, qv, y2[l]);
                }
            }
#pragma unroll
            for (int l = 0; l < N; ++l) {
                sl.Bb[l * LD + c] = bcol[l];
                sl.Qb[l * LD + c] = qcol[l];
            }
            rwarp::store_row<N>(sl.Bt + c * LD, bcol);         // row c of Bbar' = column c of Bbar
        }
        sl.sa[c] = __ldg(p.s_a + inst * N + c);                // every lane needs the whole diagonals: through the slot
        sl.ga[c] = __ldg(p.s_ga + inst * N + c);
        sl.gb[c] = __ldg(p.s_gb + inst * N + c);
        sl.gq[c] = __ldg(p.s_gq + inst * N + c);
        sl.ri[c] = __ldg(p.r_inv + inst * N + c);
        __syncwarp();
#pragma unroll 1
        for (int t = T; t >= 1; --t) {
            asm volatile("" ::: "memory");                     // the rows of Bbar, Bbar', Qbar are re-read every step, not hoisted
            const float tt = (float)t, tq = (float)(t - 1);
            float tmp[N];
            f32x2 acc[N / 2];
            zero2<N>(acc);
            mix<N>(acc, y2, sl.Bb);                            // y2 Bbar
            unpack_row<N>(tmp, acc);
#pragma unroll
            for (int l = 0; l < N; ++l) {
                const float g = __expf(-tt * sl.gb[l]);
                tmp[l] *= g * g * sl.ri[l];                    // (y3 .* g) with y3 = (y2 Bbar) .* g .* r_inv
            }
            pack_row<N>(acc, y1);
            mix<N>(acc, tmp, sl.Bt);                           // y1 + (y3 .* g) Bbar'
            unpack_row<N>(y1, acc);
            float n1 = 0.f, n2 = 0.f;
#pragma unroll
            for (int l = 0; l < N; ++l) {
                const float a = fmaf(__expf(-tt * sl.ga[l]), sl.sa[l], 1.f);
                y1[l] = __fdividef(y1[l], a);
                y2[l] *= a;
            }
            if (t >= 2) {                                      // Q_0 = 0
#pragma unroll
                for (int l = 0; l < N; ++l)
                    tmp[l] = y1[l] * __expf(-tq * sl.gq[l]);
                zero2<N>(acc);
                mix<N>(acc, tmp, sl.Qb);
                unpack_row<N>(tmp, acc);
#pragma unroll
                for (int l = 0; l < N; ++l)
                    y2[l] = fmaf(tmp[l], __expf(-tq * sl.gq[l]), y2[l]);
            }
#pragma unroll
            for (int l = 0; l < N; ++l) {
                n1 += fabsf(y1[l]);
                n2 += fabsf(y2[l]);
            }
            const float dinv = 1.f / fmaxf(fmaxf(n1, n2), 1e-30f);
#pragma unroll
            for (int l = 0; l < N; ++l) {
                y1[l] *= dinv;
                y2[l] *= dinv;
            }
        }
        // ---- Y1 P = Y2: Gauss-Jordan with partial pivoting.  Row c of [Y1 | Y2] moves to the slot (the buffers of
        // Bbar' and Qbar are free now); the pivot row is read by every lane as a broadcast.
        __syncwarp();
        float* W1 = sl.Bt;
        float* W2 = sl.Qb;
        rwarp::store_row<N>(W1 + c * LD, y1);
        rwarp::store_row<N>(W2 + c * LD, y2);
        __syncwarp();
        int my_col = -1;                                       // the column this lane's row became the pivot of
        int fail = 0;
#pragma unroll 1
        for (int j = 0; j < N; ++j) {
            const float mine = W1[c * LD + j];
            float best = (my_col < 0) ? fabsf(mine) : -1.f;
            int who = c;
#pragma unroll
            for (int o = N / 2; o > 0; o >>= 1) {
                const float ob = __shfl_xor_sync(0xffffffffu, best, o, N);
                const int ow = __shfl_xor_sync(0xffffffffu, who, o, N);
                if (ob > best || (ob == best && ow < who)) {
                    best = ob;
                    who = ow;
                }
            }
            if (!(best > 0.f) && !fail)
                fail = j + 1;
            const float piv = W1[who * LD + j];
            const float f = (c == who || !(best > 0.f)) ? 0.f : __fdividef(mine, piv);
            float pr1[N], pr2[N];
            rwarp::load_row<N>(pr1, W1 + who * LD);
            rwarp::load_row<N>(pr2, W2 + who * LD);
            rwarp::load_row<N>(y1, W1 + c * LD);
            rwarp::load_row<N>(y2, W2 + c * LD);
            __syncwarp();                                      // every lane has read the pivot row
#pragma unroll
            for (int l = 0; l < N; ++l) {
                y1[l] = fmaf(-f, pr1[l], y1[l]);
                y2[l] = fmaf(-f, pr2[l], y2[l]);
            }
            rwarp::store_row<N>(W1 + c * LD, y1);
            rwarp::store_row<N>(W2 + c * LD, y2);
            if (c == who)
                my_col = j;
            __syncwarp();
        }
        // lane with my_col = j holds row j of P_0 scaled by its pivot
        float lam = 0.f;
        {
            const float piv = my_col >= 0 ? W1[c * LD + my_col] : 1.f;
            const float pinv = 1.f / piv;
            rwarp::load_row<N>(y2, W2 + c * LD);
#pragma unroll
            for (int l = 0; l < N; ++l) {
                y2[l] *= pinv;
                lam = fmaf(y2[l], __ldg(p.h0 + inst * N + l), lam);
            }
        }
        if (p.P0 && active) {
            const float qn = quiet_nan();
            const int row = fail ? c : my_col;
#pragma unroll
            for (int l = 0; l < N; ++l)
                p.P0[inst * (long long)N * N + row * N + l] = fail ? qn : y2[l];
        }
        // lambda_0[j] sits in the lane whose row became pivot j; A_1^{-T} lambda_0 needs a_1[j] of that index
        if (my_col >= 0) {
            const float a1 = fmaf(__expf(-sl.ga[my_col]), sl.sa[my_col], 1.f);
            sl.vec[my_col] = __fdividef(lam, a1);
        }
        __syncwarp();
        {
            float w = 0.f;
#pragma unroll
            for (int k = 0; k < N; ++k)
                w = fmaf(sl.Bb[k * LD + c], sl.vec[k], w);       // (Bbar' v)[c]
            const float rc = sl.ri[c], gc = __expf(-sl.gb[c]);
            if (p.u1 && active)
                p.u1[inst * N + c] = fail ? quiet_nan() : -rc * gc * w;
        }
        if (p.info && active && c == 0)
            p.info[inst] = fail;
    }
}

template <int N>
inline size_t smem_bytes() { return sizeof(Slot<N>) * Shape<N>::SLOTS; }

} // namespace sigma
} // namespace ttc
