// Gradients of the contextualised layer's output u_1* with respect to what the coefficient layers hand over
// (Thm 3.2, then the chain rule through the Contextualization / Parameterization paragraphs), without ever forming
// the per-step matrices dA_t, dB_t, dQ_t, dR_t: every outer product of the theorem is reduced on the fly onto
// s_A, s_GammaA, s_GammaB, s_GammaQ, R^{-1}, h_0 and onto three d x d matrices per instance (the gradients of
// Bbar = sum_k s_B[k] B^(k), Qbar = sum_k s_Q[k] Q^(k) and Q_T), which are then contracted with the bases.
//
// Launches: (1) ttc_layer_kernel<N, true>: backward Riccati pass, keeps every gain K_s and k_0 = -S_0^{-1} g;
// (2) layer_grad_vectors_kernel<N>: both rollouts (primal from h_0; dual from 0 with first control k_0), both
// co-state recursions backwards, and the reductions; (3) basis_reduce_kernel: dB^(k) = sum_i s_B[i][k] dBbar_i etc.
//
// Step s = t - 1 (library indexing) uses a_s = 1 + e^{-(s+1) gA} sA (diagonal of A_{s+1}), B_s = Bbar diag(e^{-(s+1) gB}),
// R = diag(1 / r_inv), state weight Q_s = G Qbar G with G = diag(e^{-s gQ}) for s >= 1, Q_0 = 0, terminal weight Q_T.
//   dA_s[i,i] = lam_{s+1}[i] xd_s[i] + lamd_{s+1}[i] x_s[i]          -> d sA, d gA
//   dB_s      = lam_{s+1} ud_s' + lamd_{s+1} u_s'                    -> d Bbar (column-scaled), d gB
//   dQ_s      = 1/2 (x_s xd_s' + xd_s x_s')  (1 <= s <= T-1; s = T: Q_T) -> d Qbar (scaled both sides), d gQ, d Q_T
//   dR_s[j,j] = u_s[j] ud_s[j]                                        -> d r_inv = -dR / r_inv^2
//   lam_T = Q_T x_T,  lam_s = a_s .* lam_{s+1} + Q_s x_s  (same for the dual);   d h_0 = lamd_0.
// Thread mapping as in ttc_layer_kernel: N lanes per instance, lane c owns column c / component c.
#pragma once

#include "ttc_layer.cuh"

namespace ttc {
namespace lgrad {

using rwarp::Shape;
using rwarp::THREADS;
using rwarp::load_row;

struct LayerGradParams {
    layer::LayerParams lp;       // inputs; Kws, g, k0 filled by the host
    float* vec;                  // [N][4 (T + 1)][n]: x_0..x_T | xd_0..xd_T | u_0..u_{T-1}, pad | ud_0..ud_{T-1}, pad
    const int* info;             // [N]: status of the backward pass (failed instances give NaN gradients)
    float *d_sa, *d_ga, *d_gb, *d_gq, *d_ri, *d_h0;     // [N][n], each may be null
    float *d_sb, *d_sq, *d_sqf;                         // [N][r], each may be null
    float *GB, *GQ, *GF;         // [N][n][n] per-instance gradients of Bbar, Qbar, Q_T for the basis reduction, or null
};

template <int N>
struct Slot {
    float Bb[Shape<N>::MAT], Qb[Shape<N>::MAT], Qf[Shape<N>::MAT];      // rows of Bbar, Qbar, Q_T
    float x[N], xd[N], gu[N], gud[N], lam[N], lamd[N], gq[N];
};

template <int N>
__device__ __forceinline__ float seg_sum(float v)
{
#pragma unroll
    for (int o = N / 2; o > 0; o >>= 1)
        v += __shfl_xor_sync(0xffffffffu, v, o, N);
    return v;
}
// dot product of a vector in registers with a row of N floats in shared memory (the lane's own row: no conflicts)
template <int N>
__device__ __forceinline__ float dot_row(const float* row, const float (&v)[N])
{
    float acc = 0.f;
#pragma unroll
    for (int q = 0; q < N / 4; ++q) {
        const float4 r4 = *reinterpret_cast<const float4*>(row + 4 * q);
        acc = fmaf(r4.x, v[4 * q], acc);
        acc = fmaf(r4.y, v[4 * q + 1], acc);
        acc = fmaf(r4.z, v[4 * q + 2], acc);
        acc = fmaf(r4.w, v[4 * q + 3], acc);
    }
    return acc;
}
template <int N>
__device__ __forceinline__ void load_vec_global(float (&v)[N], const float* src)
{
#pragma unroll
    for (int q = 0; q < N / 4; ++q) {
        const float4 r4 = __ldg(reinterpret_cast<const float4*>(src) + q);
        v[4 * q] = r4.x; v[4 * q + 1] = r4.y; v[4 * q + 2] = r4.z; v[4 * q + 3] = r4.w;
    }
}

// the same through ordinary (coherent) loads, for data written earlier by the same kernel
template <int N>
__device__ __forceinline__ void load_vec_plain(float (&v)[N], const float* src)
{
#pragma unroll
    for (int q = 0; q < N / 4; ++q) {
        const float4 r4 = reinterpret_cast<const float4*>(src)[q];
        v[4 * q] = r4.x; v[4 * q + 1] = r4.y; v[4 * q + 2] = r4.z; v[4 * q + 3] = r4.w;
    }
}

// the kernel body is in layer_grad_body.cuh
template <int N>
__global__ void __launch_bounds__(THREADS, (N == 32) ? 2 : 4) layer_grad_vectors_kernel(LayerGradParams q);

// dBasis[k][e] += sum over a slice of instances of coef[i][k] * G[i][e]; one CTA per slice, atomics at the end.
// Up to two (coefficient, matrix) pairs go to the same destination (Q^(k) collects s_Q[k] dQbar and s_Qf[k] dQ_T).
__global__ void __launch_bounds__(256) basis_reduce_kernel(long long N, int r, int nn, const int* info,
                                                           const float* c0, const float* G0, const float* c1, const float* G1,
                                                           float* dst)
{
    constexpr int RK = 16;
    const long long per = (N + gridDim.x - 1) / gridDim.x;
    const long long i0 = per * blockIdx.x, i1 = i0 + per < N ? i0 + per : N;
    for (int e = threadIdx.x; e < nn; e += blockDim.x)
        for (int kb = 0; kb < r; kb += RK) {
            float acc[RK];
#pragma unroll
            for (int k = 0; k < RK; ++k)
                acc[k] = 0.f;
            for (long long i = i0; i < i1; ++i) {
                if (info[i] != 0)
                    continue;                                  // a failed instance contributes nothing to the shared bases
                const float v0 = G0[i * nn + e];
                const float v1 = G1 ? G1[i * nn + e] : 0.f;
#pragma unroll
                for (int k = 0; k < RK; ++k)
                    if (kb + k < r) {
                        acc[k] = fmaf(__ldg(c0 + i * r + kb + k), v0, acc[k]);
                        if (G1)
                            acc[k] = fmaf(__ldg(c1 + i * r + kb + k), v1, acc[k]);
                    }
            }
#pragma unroll
            for (int k = 0; k < RK; ++k)
                if (kb + k < r)
                    atomicAdd(dst + (long long)(kb + k) * nn + e, acc[k]);
        }
}

} // namespace lgrad
} // namespace ttc

#include "layer_grad_body.cuh"
