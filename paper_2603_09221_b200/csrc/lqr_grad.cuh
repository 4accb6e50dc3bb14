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
    int vec4;              // 1: n/4 and m/4 are powers of two and A, B are float4-addressable at every (instance, t)
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

// y[r] = sum_j M[r][j] v[j] for two vectors v, vd at once.  M: rows x cols, row-major, 16-byte aligned, cols / 4 a
// power of two <= 32; v, vd in shared memory.  The warp reads M as consecutive float4s (coalesced); the cols / 4 lanes
// that share a row add their partial sums by shuffles and the first of them hands (r, y[r], yd[r]) to `sink`.
template <typename Sink>
__device__ __forceinline__ void row_matvec2(const float* M, int rows, int cols, const float* v, const float* vd,
                                            int lane, Sink&& sink)
{
    const int q = cols >> 2, total = rows * q;
    for (int base = 0; base < total; base += 32) {
        const int e = base + lane, qc = e & (q - 1);
        float a = 0.f, ad = 0.f;
        if (e < total) {
            const float4 k = __ldg(reinterpret_cast<const float4*>(M) + e);
            const float4 x4 = *reinterpret_cast<const float4*>(v + 4 * qc);
            const float4 d4 = *reinterpret_cast<const float4*>(vd + 4 * qc);
            a = fmaf(k.x, x4.x, fmaf(k.y, x4.y, fmaf(k.z, x4.z, k.w * x4.w)));
            ad = fmaf(k.x, d4.x, fmaf(k.y, d4.y, fmaf(k.z, d4.z, k.w * d4.w)));
        }
        for (int off = 1; off < q; off <<= 1) {
            a += __shfl_xor_sync(0xffffffffu, a, off);
            ad += __shfl_xor_sync(0xffffffffu, ad, off);
        }
        if (e < total && qc == 0)
            sink(e / q, a, ad);
    }
}

// a += sum_i M[i][c] v[i], ad += sum_i M[i][c] vd[i]: column c of a row-major matrix with `ld` columns (lanes over c:
// coalesced).  The loads go out eight at a time so that their latencies overlap.
__device__ __forceinline__ void col_matvec2(const OperandDev& o, long long off, int rows, int ld, int c,
                                            const float* v, const float* vd, float& a, float& ad)
{
    for (int i0 = 0; i0 < rows; i0 += 8) {
        float mv[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
            mv[k] = (i0 + k < rows) ? load_elem(o, off + (long long)(i0 + k) * ld + c) : 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (i0 + k < rows) {
                a = fmaf(mv[k], v[i0 + k], a);
                ad = fmaf(mv[k], vd[i0 + k], ad);
            }
    }
}

__global__ void __launch_bounds__(32 * WARPS) grad_vectors_kernel(GradParams g)
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
            if (g.vec4) {
                const float* k0 = g.kff + inst * (long long)H * m;
                float* ur = vec_row(g, inst, 2, t);
                float* udr = vec_row(g, inst, 3, t);
                row_matvec2(Kt, m, n, x, xd, lane, [&](int r, float a, float ad) {
                    if (t == 0) {
                        ad += k0[r];
                        if (g.u0)
                            g.u0[inst * m + r] = a;
                    }
                    u[r] = a;
                    ud[r] = ad;
                    ur[r] = a;
                    udr[r] = ad;
                });
                const float* At = reinterpret_cast<const float*>(p.A.ptr) + oa + t * p.A.st;
                const float* Bt = reinterpret_cast<const float*>(p.B.ptr) + ob + t * p.B.st;
                row_matvec2(At, n, n, x, xd, lane, [&](int r, float a, float ad) {
                    l[r] = a;                                 // l, ld are free until the co-state loop
                    ld[r] = ad;
                });
                __syncwarp();                                 // u_t, A_t x_t complete; x_t consumed
                float* xr = vec_row(g, inst, 0, t + 1);
                float* xdr = vec_row(g, inst, 1, t + 1);
                row_matvec2(Bt, n, m, u, ud, lane, [&](int r, float a, float ad) {
                    a += l[r];
                    ad += ld[r];
                    x[r] = a;
                    xd[r] = ad;
                    xr[r] = a;
                    xdr[r] = ad;
                });
                __syncwarp();
                continue;
            }
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
                col_matvec2(F, of, n, n, c, x, xd, a, ad);    // Qf symmetric
                l[c] = a;
                ld[c] = ad;
                vec_row(g, inst, 4, H)[c] = a;
                vec_row(g, inst, 5, H)[c] = ad;
            }
        }
        __syncwarp();
        for (int t = H - 1; t >= 0; --t) {
            const long long at = oa + t * p.A.st, qt = oq + t * p.Q.st;
            float ln[2] = {0.f, 0.f}, ldn[2] = {0.f, 0.f};
#pragma unroll
            for (int h = 0; h < 2; ++h) {                     // (A_t' lam_{t+1})[c]: needs nothing of x_t
                const int c = lane + 32 * h;
                if (c < n)
                    col_matvec2(p.A, at, n, n, c, l, ld, ln[h], ldn[h]);
            }
            for (int c = lane; c < n; c += 32) {              // own stores of the forward loop
                x[c] = vec_row(g, inst, 0, t)[c];
                xd[c] = vec_row(g, inst, 1, t)[c];
            }
            __syncwarp();
#pragma unroll
            for (int h = 0; h < 2; ++h) {                     // + (Q_t x_t)[c], Q_t symmetric
                const int c = lane + 32 * h;
                if (c < n)
                    col_matvec2(p.Q, qt, n, n, c, x, xd, ln[h], ldn[h]);
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

// ---- n, m <= 16 (the layer's own sizes).  The recurrences are sequential in t and every step needs a few KB that
// no earlier step produced (K_t, A_t, B_t forward; A_t, Q_t, x_t backward), so the kernel is bound by memory latency
// unless those bytes are requested several steps ahead: each warp keeps a ring of STAGES steps in shared memory,
// filled by 16-byte cp.async copies (every matrix of a step is at most two float4 per lane).

constexpr int STAGES = 4;

struct __align__(16) Stage {
    float4 K[64];          // K_t (forward) or Q_t (backward)
    float4 A[64];
    float4 B[64];
    float xv[16], xdv[16]; // x_t, xd_t (backward)
};

struct Mat2 { float4 v[2]; };

__device__ __forceinline__ void cp16(void* dst_smem, const void* src)
{
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst_smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }

__device__ __forceinline__ void stage_mat(float4* dst, const float* src, int total, int lane)
{
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int e = 32 * k + lane;
        if (e < total)
            cp16(dst + e, src + 4 * e);
    }
}

__device__ __forceinline__ void read_mat2(Mat2& d, const float4* src, int total, int lane)
{
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int e = 32 * k + lane;
        d.v[k] = e < total ? src[e] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
}

// y[r] = sum_j M[r][j] v[j] (two vectors), M held as float4 number e = lane + 32 k of a rows x (4 q) matrix; x4, d4
// are the lane's own four elements of v and vd: v[4 qc .. 4 qc + 3] with qc = lane & (q - 1)
template <typename Sink>
__device__ __forceinline__ void row_mv_reg(const Mat2& M, int rows, int q, int lq, const float4 x4, const float4 d4,
                                           int lane, Sink&& sink)
{
    const int total = rows * q;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        if (32 * k >= total)
            break;
        const int e = 32 * k + lane, qc = e & (q - 1);
        const float4 m4 = M.v[k];
        float a = fmaf(m4.x, x4.x, fmaf(m4.y, x4.y, fmaf(m4.z, x4.z, m4.w * x4.w)));
        float ad = fmaf(m4.x, d4.x, fmaf(m4.y, d4.y, fmaf(m4.z, d4.z, m4.w * d4.w)));
        for (int off = 1; off < q; off <<= 1) {
            a += __shfl_xor_sync(0xffffffffu, a, off);
            ad += __shfl_xor_sync(0xffffffffu, ad, off);
        }
        if (e < total && qc == 0)
            sink(e >> lq, a, ad);
    }
}

// y[c] = sum_i M[i][c] v[i] (two vectors), same register layout; lanes 0..q-1 end up with columns 4 lane .. 4 lane + 3
template <typename Sink>
__device__ __forceinline__ void col_mv_reg(const Mat2& M, int rows, int q, int lq, const float* v, const float* vd,
                                           int lane, Sink&& sink)
{
    const int total = rows * q;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), ad = a;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int e = 32 * k + lane;
        if (e < total) {
            const float vi = v[e >> lq], di = vd[e >> lq];
            const float4 m4 = M.v[k];
            a.x = fmaf(m4.x, vi, a.x); a.y = fmaf(m4.y, vi, a.y); a.z = fmaf(m4.z, vi, a.z); a.w = fmaf(m4.w, vi, a.w);
            ad.x = fmaf(m4.x, di, ad.x); ad.y = fmaf(m4.y, di, ad.y); ad.z = fmaf(m4.z, di, ad.z); ad.w = fmaf(m4.w, di, ad.w);
        }
    }
    for (int off = q; off < 32; off <<= 1) {
        a.x += __shfl_xor_sync(0xffffffffu, a.x, off); a.y += __shfl_xor_sync(0xffffffffu, a.y, off);
        a.z += __shfl_xor_sync(0xffffffffu, a.z, off); a.w += __shfl_xor_sync(0xffffffffu, a.w, off);
        ad.x += __shfl_xor_sync(0xffffffffu, ad.x, off); ad.y += __shfl_xor_sync(0xffffffffu, ad.y, off);
        ad.z += __shfl_xor_sync(0xffffffffu, ad.z, off); ad.w += __shfl_xor_sync(0xffffffffu, ad.w, off);
    }
    if (lane < q)
        sink(4 * lane, a, ad);
}

inline size_t small_smem_bytes() { return WARPS * (STAGES * sizeof(Stage) + 6 * 16 * sizeof(float)); }

// Requires: n, m in {4, 8, 16}; A, B, Q, Qf float32 and float4-addressable at every (instance, t).
__global__ void __launch_bounds__(32 * WARPS) grad_vectors_small_kernel(GradParams g)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const SolveParams& p = g.sp;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = p.n, m = p.m, H = p.H;
    Stage* ring = reinterpret_cast<Stage*>(smem_raw) + warp * STAGES;
    float* vecs = reinterpret_cast<float*>(smem_raw + WARPS * STAGES * sizeof(Stage)) + warp * 6 * 16;
    float* x = vecs;
    float* xd = vecs + 16;
    float* u = vecs + 32;
    float* ud = vecs + 48;
    float* l = vecs + 64;
    float* ld = vecs + 80;
    const int qn = n >> 2, qm = m >> 2, lqn = 31 - __clz(qn), lqm = 31 - __clz(qm);
    const int tK = m * qn, tA = n * qn, tB = n * qm;          // float4s per matrix

    for (long long inst = (long long)blockIdx.x * WARPS + warp; inst < p.N; inst += (long long)gridDim.x * WARPS) {
        const float* Ab = reinterpret_cast<const float*>(p.A.ptr) + operand_offset(p.A, inst, p.b1, p.b2);
        const float* Bb = reinterpret_cast<const float*>(p.B.ptr) + operand_offset(p.B, inst, p.b1, p.b2);
        const float* Qb = reinterpret_cast<const float*>(p.Q.ptr) + operand_offset(p.Q, inst, p.b1, p.b2);
        const float* Fb = p.Qf.ptr ? reinterpret_cast<const float*>(p.Qf.ptr) + operand_offset(p.Qf, inst, p.b1, p.b2)
                                   : Qb;
        const float* Kb = g.K + inst * (long long)H * m * n;
        const float* k0 = g.kff + inst * (long long)H * m;

        auto issue_fwd = [&](int t) {                         // one commit group per step, also past the end
            if (t < H) {
                Stage& s = ring[t % STAGES];
                stage_mat(s.K, Kb + (long long)t * m * n, tK, lane);
                stage_mat(s.A, Ab + t * p.A.st, tA, lane);
                stage_mat(s.B, Bb + t * p.B.st, tB, lane);
            }
            cp_commit();
        };
        auto issue_bwd = [&](int t) {
            if (t >= 0) {
                Stage& s = ring[t % STAGES];
                stage_mat(s.K, Qb + t * p.Q.st, tA, lane);
                stage_mat(s.A, Ab + t * p.A.st, tA, lane);
                if (lane < qn) {
                    cp16(s.xv + 4 * lane, vec_row(g, inst, 0, t) + 4 * lane);
                    cp16(s.xdv + 4 * lane, vec_row(g, inst, 1, t) + 4 * lane);
                }
            }
            cp_commit();
        };

        __syncwarp();                                         // the previous instance is done with the ring
#pragma unroll
        for (int t = 0; t < STAGES - 1; ++t)
            issue_fwd(t);
        Mat2 fq;
        {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int e = 32 * k + lane;
                fq.v[k] = e < tA ? __ldg(reinterpret_cast<const float4*>(Fb) + e) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        const float xd0 = isnan(Kb[0]) ? quiet_nan() : 0.f;   // failed backward pass: every gradient NaN
        if (lane < n) {
            const float v = load_elem(p.x0, operand_offset(p.x0, inst, p.b1, p.b2) + lane);
            x[lane] = v;
            xd[lane] = xd0;
            vec_row(g, inst, 0, 0)[lane] = v;
            vec_row(g, inst, 1, 0)[lane] = xd0;
        }

        for (int t = 0; t < H; ++t) {
            issue_fwd(t + STAGES - 1);                        // its slot was read in step t - 1
            cp_wait<STAGES - 1>();                            // this lane's copies of step t have landed
            __syncwarp();                                     // ... and every other lane's; x_t is complete
            const Stage& s = ring[t % STAGES];
            Mat2 kq, aq, bq;
            read_mat2(kq, s.K, tK, lane);
            read_mat2(aq, s.A, tA, lane);
            read_mat2(bq, s.B, tB, lane);
            float* ur = vec_row(g, inst, 2, t);
            float* udr = vec_row(g, inst, 3, t);
            const float4 x4 = *reinterpret_cast<const float4*>(x + 4 * (lane & (qn - 1)));
            const float4 xd4 = *reinterpret_cast<const float4*>(xd + 4 * (lane & (qn - 1)));
            row_mv_reg(kq, m, qn, lqn, x4, xd4, lane, [&](int r, float a, float ad) {
                if (t == 0) {
                    ad += k0[r];
                    if (g.u0)
                        g.u0[inst * m + r] = a;
                }
                u[r] = a;
                ud[r] = ad;
                ur[r] = a;
                udr[r] = ad;
            });
            row_mv_reg(aq, n, qn, lqn, x4, xd4, lane, [&](int r, float a, float ad) {
                l[r] = a;                                     // l, ld are free until the co-state loop
                ld[r] = ad;
            });
            __syncwarp();
            float* xr = vec_row(g, inst, 0, t + 1);
            float* xdr = vec_row(g, inst, 1, t + 1);
            const float4 u4 = *reinterpret_cast<const float4*>(u + 4 * (lane & (qm - 1)));
            const float4 ud4 = *reinterpret_cast<const float4*>(ud + 4 * (lane & (qm - 1)));
            row_mv_reg(bq, n, qm, lqm, u4, ud4, lane, [&](int r, float a, float ad) {
                a += l[r];
                ad += ld[r];
                x[r] = a;
                xd[r] = ad;
                xr[r] = a;
                xdr[r] = ad;
            });
        }
        cp_wait<0>();
        __syncwarp();                                         // x_H complete; every x_t, xd_t of this warp is ordered before the copies below

        // ---- co-states.  lam_H = Qf x_H (Qf symmetric: row form)
#pragma unroll
        for (int j = 0; j < STAGES - 1; ++j)
            issue_bwd(H - 1 - j);
        {
            float* lr = vec_row(g, inst, 4, H);
            float* ldr = vec_row(g, inst, 5, H);
            const float4 x4 = *reinterpret_cast<const float4*>(x + 4 * (lane & (qn - 1)));
            const float4 xd4 = *reinterpret_cast<const float4*>(xd + 4 * (lane & (qn - 1)));
            row_mv_reg(fq, n, qn, lqn, x4, xd4, lane, [&](int r, float a, float ad) {
                l[r] = a;
                ld[r] = ad;
                lr[r] = a;
                ldr[r] = ad;
            });
        }
        for (int t = H - 1; t >= 0; --t) {
            cp_wait<STAGES - 2>();                            // this lane's copies of step t have landed
            __syncwarp();                                     // ... and every other lane's; lam_{t+1} complete
            issue_bwd(t - (STAGES - 1));                      // its slot (x_{t+1} included) was read in step t + 1
            const Stage& s = ring[t % STAGES];
            Mat2 aq, qq;
            read_mat2(aq, s.A, tA, lane);
            read_mat2(qq, s.K, tA, lane);
            col_mv_reg(aq, n, qn, lqn, l, ld, lane, [&](int c0, const float4& a, const float4& ad) {     // A_t' lam_{t+1}
                *reinterpret_cast<float4*>(u + c0) = a;
                *reinterpret_cast<float4*>(ud + c0) = ad;
            });
            __syncwarp();
            float* lr = vec_row(g, inst, 4, t);
            float* ldr = vec_row(g, inst, 5, t);
            const float4 x4 = *reinterpret_cast<const float4*>(s.xv + 4 * (lane & (qn - 1)));
            const float4 xd4 = *reinterpret_cast<const float4*>(s.xdv + 4 * (lane & (qn - 1)));
            row_mv_reg(qq, n, qn, lqn, x4, xd4, lane, [&](int r, float a, float ad) {                    // + Q_t x_t
                a += u[r];
                ad += ud[r];
                l[r] = a;
                ld[r] = ad;
                lr[r] = a;
                ldr[r] = ad;
                if (t == 0 && g.dx0)
                    g.dx0[inst * n + r] = ad;
            });
        }
        cp_wait<0>();
    }
}

// dst[r][c] = scale * (a1[r] b1[c] + a2[r] b2[c]),  rows x cols, row-major, written by one warp.  Each product is
// rounded before the sum (no fused multiply-add), so the symmetric outputs (a2 = b1, b2 = a1, scale a power of two)
// come out bit-symmetric.
__device__ __forceinline__ void emit_outer(float* dst, int rows, int cols, const float* a1, const float* b1,
                                           const float* a2, const float* b2, float scale, int lane)
{
    if ((cols & 3) == 0 && ((cols >> 2) & ((cols >> 2) - 1)) == 0 && cols <= 64) {
        // cols / 4 a power of two <= 16: a lane keeps its four columns for every row it writes
        const int c4n = cols >> 2, lc = 31 - __clz(c4n), rstep = 32 >> lc;
        const int c = (lane & (c4n - 1)) * 4;
        const float4 v1 = *reinterpret_cast<const float4*>(b1 + c);
        const float4 v2 = *reinterpret_cast<const float4*>(b2 + c);
        float4* d4 = reinterpret_cast<float4*>(dst) + lane;
        for (int r = lane >> lc; r < rows; r += rstep, d4 += 32) {
            const float p1 = scale * a1[r], p2 = scale * a2[r];
            float4 o;
            o.x = __fadd_rn(__fmul_rn(p1, v1.x), __fmul_rn(p2, v2.x));
            o.y = __fadd_rn(__fmul_rn(p1, v1.y), __fmul_rn(p2, v2.y));
            o.z = __fadd_rn(__fmul_rn(p1, v1.z), __fmul_rn(p2, v2.z));
            o.w = __fadd_rn(__fmul_rn(p1, v1.w), __fmul_rn(p2, v2.w));
            __stcs(d4, o);                                    // written once, never re-read here
        }
    } else if ((cols & 3) == 0) {
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
    const long long stride = (long long)gridDim.x * WARPS;
    const bool small_items = items < (1ll << 31);             // 32-bit division is several times cheaper
    long long it = (long long)blockIdx.x * WARPS + warp;

    // the six vectors of one item, two elements per lane; fetched one item ahead of the stores
    float rv[6][2];
    auto fetch = [&](long long item) {
        const long long inst = small_items ? (long long)((unsigned)item / (unsigned)(H + 1)) : item / (H + 1);
        const int t = (int)(item - inst * (H + 1));
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int c = lane + 32 * h;
            const bool cn = c < n, cm = c < m && t < H;
            rv[0][h] = cn ? vec_row(g, inst, 0, t)[c] : 0.f;
            rv[1][h] = cn ? vec_row(g, inst, 1, t)[c] : 0.f;
            rv[2][h] = cm ? vec_row(g, inst, 2, t)[c] : 0.f;
            rv[3][h] = cm ? vec_row(g, inst, 3, t)[c] : 0.f;
            rv[4][h] = (cn && t < H) ? vec_row(g, inst, 4, t + 1)[c] : 0.f;
            rv[5][h] = (cn && t < H) ? vec_row(g, inst, 5, t + 1)[c] : 0.f;
        }
    };
    if (it < items)
        fetch(it);
    while (it < items) {
        const long long inst = small_items ? (long long)((unsigned)it / (unsigned)(H + 1)) : it / (H + 1);
        const int t = (int)(it - inst * (H + 1));
        __syncwarp();                                         // the previous item's reads of shared memory are done
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int c = lane + 32 * h;
            x[c] = rv[0][h];
            xd[c] = rv[1][h];
            u[c] = rv[2][h];
            ud[c] = rv[3][h];
            l[c] = rv[4][h];
            ld[c] = rv[5][h];
        }
        __syncwarp();
        const long long nx = it + stride;
        if (nx < items)
            fetch(nx);                                        // in flight while this item's rows are written
        if (t == H) {
            if (g.dQf)
                emit_outer(g.dQf + inst * (long long)n * n, n, n, x, xd, xd, x, 0.5f, lane);
        } else {
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
        it = nx;
    }
}

} // namespace grad
} // namespace ttc
