// Gradients of the layer output u_0* (Thm 3.2), after the backward Riccati pass has left K_t and k_0.
//
// Two kernels:
//  * grad_vectors_kernel  -- one warp per instance: primal rollout x_t, u_t (u_t = K_t x_t), dual rollout
//    xd_t, ud_t (xd_0 = 0, ud_0 = k_0 = -S_0^{-1} g, then ud_t = K_t xd_t: the dual problem's linear cost sits on
//    the first control only, so p_t = 0 and k_t = 0 for t >= 1), and the co-states of both by the backward relation
//    lam_H = Qf x_H, lam_t = A_t' lam_{t+1} + Q_t x_t.  The six vector sequences go to a workspace.
//  * grad_outer_kernel    -- one warp per (instance, t): the outer products of Thm 3.2, streamed out as rows.
//    This is the kernel that writes almost all of the bytes: 2 n^2 + n m + m^2 floats per (instance, t).
//
// Q_t and Qf are taken as symmetric (the co-state products read them by columns).
#pragma once
#include "common.cuh"

namespace ttc {
namespace grad {

constexpr int WARPS = 8;
constexpr int DMAX = 64;

struct GradParams {
    SolveParams sp;        // operands, batch, n, m, H
    const float* K;        // [N][H][m][n]
    const float* kff;      // [N][H][m]   (only t = 0 is read)
    float* vec;            // [N][6][H+1][D]: x, xd, u, ud, lam, lamd
    int D;                 // row length of vec: max(n, m) rounded up to a multiple of 4
    float* dA;             // [N][H][n][n] or null
    float* dB;             // [N][H][n][m] or null
    float* dQ;             // [N][H][n][n] or null
    float* dQf;            // [N][n][n] or null
    float* dR;             // [N][H][m][m] or null
    float* dx0;            // [N][n] or null
    float* u0;             // [N][m] or null
};

__device__ __forceinline__ float* vec_row(const GradParams& g, long long inst, int which, int t)
{
    return g.vec + ((inst * 6 + which) * (long long)(g.sp.H + 1) + t) * g.D;
}

__global__ void __launch_bounds__(32 * WARPS) grad_vectors_kernel(GradParams g)
{
    __shared__ float sm[WARPS][6][DMAX];
    const SolveParams& p = g.sp;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = p.n, m = p.m, H = p.H;
    float* x = sm[warp][0];
    float* xd = sm[warp][1];
    float* u = sm[warp][2];
    float* ud = sm[warp][3];
    float* l = sm[warp][4];
    float* ld = sm[warp][5];
    const bool k4 = (n & 3) == 0;                             // rows of K_t are float4-addressable

    for (long long inst = (long long)blockIdx.x * WARPS + warp; inst < p.N; inst += (long long)gridDim.x * WARPS) {
        const long long oa = operand_offset(p.A, inst, p.b1, p.b2);
        const long long ob = operand_offset(p.B, inst, p.b1, p.b2);
        const long long oq = operand_offset(p.Q, inst, p.b1, p.b2);
        // a failed backward pass left quiet NaNs in K: make every gradient of that instance NaN, also the
        // products with xd_0 = 0
        const float xd0 = isnan(g.K[inst * (long long)H * m * n]) ? quiet_nan() : 0.f;
        for (int c = lane; c < n; c += 32) {
            const float v = load_elem(p.x0, operand_offset(p.x0, inst, p.b1, p.b2) + c);
            x[c] = v;
            xd[c] = xd0;
            vec_row(g, inst, 0, 0)[c] = v;
            vec_row(g, inst, 1, 0)[c] = xd0;
        }
        __syncwarp();

        // ---- forward: both rollouts share every load of K_t, A_t, B_t
        for (int t = 0; t < H; ++t) {
            const float* Kt = g.K + (inst * (long long)H + t) * m * n;
            for (int c = lane; c < m; c += 32) {
                float a = 0.f, ad = (t == 0) ? g.kff[inst * (long long)H * m + c] : 0.f;
                if (k4) {
                    const float4* kr = reinterpret_cast<const float4*>(Kt + (long long)c * n);
                    for (int q = 0; q < n / 4; ++q) {
                        const float4 k = kr[q];
                        a = fmaf(k.x, x[4 * q], a);         ad = fmaf(k.x, xd[4 * q], ad);
                        a = fmaf(k.y, x[4 * q + 1], a);     ad = fmaf(k.y, xd[4 * q + 1], ad);
                        a = fmaf(k.z, x[4 * q + 2], a);     ad = fmaf(k.z, xd[4 * q + 2], ad);
                        a = fmaf(k.w, x[4 * q + 3], a);     ad = fmaf(k.w, xd[4 * q + 3], ad);
                    }
                } else {
                    for (int j = 0; j < n; ++j) {
                        const float k = Kt[c * n + j];
                        a = fmaf(k, x[j], a);
                        ad = fmaf(k, xd[j], ad);
                    }
                }
                u[c] = a;
                ud[c] = ad;
                vec_row(g, inst, 2, t)[c] = a;
                vec_row(g, inst, 3, t)[c] = ad;
                if (t == 0 && g.u0)
                    g.u0[inst * m + c] = a;
            }
            __syncwarp();
            const long long at = oa + t * p.A.st, bt = ob + t * p.B.st;
            float xn[2] = {0.f, 0.f}, xdn[2] = {0.f, 0.f};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = lane + 32 * h;
                if (c < n) {
                    float a = 0.f, ad = 0.f;
                    for (int j = 0; j < n; ++j) {
                        const float v = load_elem(p.A, at + (long long)c * n + j);
                        a = fmaf(v, x[j], a);
                        ad = fmaf(v, xd[j], ad);
                    }
                    for (int j = 0; j < m; ++j) {
                        const float v = load_elem(p.B, bt + (long long)c * m + j);
                        a = fmaf(v, u[j], a);
                        ad = fmaf(v, ud[j], ad);
                    }
                    xn[h] = a;
                    xdn[h] = ad;
                }
            }
            __syncwarp();                                     // x_t consumed by every lane
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = lane + 32 * h;
                if (c < n) {
                    x[c] = xn[h];
                    xd[c] = xdn[h];
                    vec_row(g, inst, 0, t + 1)[c] = xn[h];
                    vec_row(g, inst, 1, t + 1)[c] = xdn[h];
                }
            }
            __syncwarp();
        }

        // ---- co-states, backward.  x, xd hold x_H, xd_H.
        {
            const OperandDev& F = p.Qf.ptr ? p.Qf : p.Q;
            const long long of = operand_offset(F, inst, p.b1, p.b2);
            for (int c = lane; c < n; c += 32) {
                float a = 0.f, ad = 0.f;
                for (int j = 0; j < n; ++j) {
                    const float v = load_elem(F, of + (long long)j * n + c);
                    a = fmaf(v, x[j], a);
                    ad = fmaf(v, xd[j], ad);
                }
                l[c] = a;
                ld[c] = ad;
                vec_row(g, inst, 4, H)[c] = a;
                vec_row(g, inst, 5, H)[c] = ad;
            }
        }
        __syncwarp();
        for (int t = H - 1; t >= 0; --t) {
            for (int c = lane; c < n; c += 32) {              // own stores of the forward loop
                x[c] = vec_row(g, inst, 0, t)[c];
                xd[c] = vec_row(g, inst, 1, t)[c];
            }
            __syncwarp();
            const long long at = oa + t * p.A.st, qt = oq + t * p.Q.st;
            float ln[2] = {0.f, 0.f}, ldn[2] = {0.f, 0.f};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = lane + 32 * h;
                if (c < n) {
                    float a = 0.f, ad = 0.f;
                    for (int i = 0; i < n; ++i) {
                        const float av = load_elem(p.A, at + (long long)i * n + c);     // (A_t' lam)[c]
                        const float qv = load_elem(p.Q, qt + (long long)i * n + c);     // (Q_t x)[c], Q_t symmetric
                        a = fmaf(av, l[i], fmaf(qv, x[i], a));
                        ad = fmaf(av, ld[i], fmaf(qv, xd[i], ad));
                    }
                    ln[h] = a;
                    ldn[h] = ad;
                }
            }
            __syncwarp();
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = lane + 32 * h;
                if (c < n) {
                    l[c] = ln[h];
                    ld[c] = ldn[h];
                    vec_row(g, inst, 4, t)[c] = ln[h];
                    vec_row(g, inst, 5, t)[c] = ldn[h];
                    if (t == 0 && g.dx0)
                        g.dx0[inst * n + c] = ldn[h];
                }
            }
            __syncwarp();
        }
    }
}

// dst[r][c] = scale * (a1[r] b1[c] + a2[r] b2[c]),  rows x cols, row-major, written by one warp.  Each product is
// rounded before the sum (no fused multiply-add), so the symmetric outputs (a2 = b1, b2 = a1, scale a power of two)
// come out bit-symmetric.
__device__ __forceinline__ void emit_outer(float* dst, int rows, int cols, const float* a1, const float* b1,
                                           const float* a2, const float* b2, float scale, int lane)
{
    if ((cols & 3) == 0) {
        const int c4n = cols >> 2, cnt = rows * c4n;
        float4* d4 = reinterpret_cast<float4*>(dst);
        for (int e = lane; e < cnt; e += 32) {
            const int r = e / c4n, c = (e - r * c4n) * 4;
            const float p1 = scale * a1[r], p2 = scale * a2[r];
            const float4 v1 = *reinterpret_cast<const float4*>(b1 + c);
            const float4 v2 = *reinterpret_cast<const float4*>(b2 + c);
            float4 o;
            o.x = __fadd_rn(__fmul_rn(p1, v1.x), __fmul_rn(p2, v2.x));
            o.y = __fadd_rn(__fmul_rn(p1, v1.y), __fmul_rn(p2, v2.y));
            o.z = __fadd_rn(__fmul_rn(p1, v1.z), __fmul_rn(p2, v2.z));
            o.w = __fadd_rn(__fmul_rn(p1, v1.w), __fmul_rn(p2, v2.w));
            __stcs(d4 + e, o);                                // written once, never re-read here
        }
    } else {
        const int cnt = rows * cols;
        for (int e = lane; e < cnt; e += 32) {
            const int r = e / cols, c = e - r * cols;
            dst[e] = __fadd_rn(__fmul_rn(scale * a1[r], b1[c]), __fmul_rn(scale * a2[r], b2[c]));
        }
    }
}

__global__ void __launch_bounds__(32 * WARPS) grad_outer_kernel(GradParams g)
{
    __shared__ __align__(16) float sm[WARPS][6][DMAX];
    const SolveParams& p = g.sp;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = p.n, m = p.m, H = p.H;
    float* x = sm[warp][0];
    float* xd = sm[warp][1];
    float* u = sm[warp][2];
    float* ud = sm[warp][3];
    float* l = sm[warp][4];
    float* ld = sm[warp][5];
    const long long items = p.N * (long long)(H + 1);
    for (long long it = (long long)blockIdx.x * WARPS + warp; it < items; it += (long long)gridDim.x * WARPS) {
        const long long inst = it / (H + 1);
        const int t = (int)(it - inst * (H + 1));
        __syncwarp();
        for (int c = lane; c < n; c += 32) {
            x[c] = vec_row(g, inst, 0, t)[c];
            xd[c] = vec_row(g, inst, 1, t)[c];
            if (t < H) {
                l[c] = vec_row(g, inst, 4, t + 1)[c];
                ld[c] = vec_row(g, inst, 5, t + 1)[c];
            }
        }
        if (t < H)
            for (int c = lane; c < m; c += 32) {
                u[c] = vec_row(g, inst, 2, t)[c];
                ud[c] = vec_row(g, inst, 3, t)[c];
            }
        __syncwarp();
        if (t == H) {
            if (g.dQf)
                emit_outer(g.dQf + inst * (long long)n * n, n, n, x, xd, xd, x, 0.5f, lane);
            continue;
        }
        const long long step = inst * (long long)H + t;
        if (g.dA)
            emit_outer(g.dA + step * n * n, n, n, l, xd, ld, x, 1.f, lane);
        if (g.dB)
            emit_outer(g.dB + step * n * m, n, m, l, ud, ld, u, 1.f, lane);
        if (g.dQ)
            emit_outer(g.dQ + step * n * n, n, n, x, xd, xd, x, 0.5f, lane);
        if (g.dR)
            emit_outer(g.dR + step * m * m, m, m, u, ud, ud, u, 0.5f, lane);
    }
}

} // namespace grad
} // namespace ttc
