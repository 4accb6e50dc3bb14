// Shared device-side definitions of the LQR kernels: launch parameters, operand
// addressing (batch strides with broadcast), element loads with bf16 widening.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ttc_lqr.h"

namespace ttc {

struct OperandDev {
    const void* ptr;
    int dtype;            // TTC_F32 | TTC_BF16
    long long s0, s1, s2; // element strides of the three batch dimensions (0 = shared)
    long long st;         // element stride between consecutive time indices (0 = the same matrix at every t)
};

struct SolveParams {
    int n, m, H;
    long long b0, b1, b2, N;   // batch dims and their product
    long long t0, tcount;      // token window [t0, t0 + tcount) of the last batch dimension solved by this launch
    OperandDev A, B, Q, R, x0;
    OperandDev Qf;             // terminal weight P_H (ptr null: P_H = Q)
    OperandDev r;              // linear control cost r_t (vector of m; ptr null: none), Prop. A.1
    int r_count;               // r_t is given for t < r_count and zero from there on (the dual problem of Thm 3.2 has r_0 only)
    float* K;      // [N][H][m][n] or null
    float* P;      // [N][H+1][n][n] ([N][n][n] when first_only) or null
    float* x;      // [N][H+1][n] or null
    float* u;      // [N][H][m] ([N][m] when first_only) or null
    int* info;     // [N] or null
    float* Kws;    // workspace gains [N][H][m][n]: used when the rollout needs K_t but K is null
    float* kff;    // feed-forward terms k_t [N][H][m] (caller's output or workspace) when r is given, else null
    float* pvec;   // p_t [N][H+1][n] ([N][n] when first_only) or null
    int first_only;
    int out_bf16;  // K, P, x, u are bfloat16 arrays (round to nearest even) instead of float32
};

__device__ __forceinline__ long long operand_offset(const OperandDev& o, long long i, long long b1,
                                                    long long b2)
{
    long long i2 = i % b2;
    long long r = i / b2;
    long long i1 = r % b1;
    long long i0 = r / b1;
    return i0 * o.s0 + i1 * o.s1 + i2 * o.s2;
}

// w-th instance of the launch's token window (w in [0, b0 * b1 * tcount)) -> instance index
__device__ __forceinline__ long long window_instance(const SolveParams& p, long long w)
{
    return (w / p.tcount) * p.b2 + p.t0 + w % p.tcount;
}

__device__ __forceinline__ float load_elem(const OperandDev& o, long long idx)
{
    if (o.dtype == TTC_BF16)
        return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(o.ptr)[idx]);
    return reinterpret_cast<const float*>(o.ptr)[idx];
}

// Copy `cnt` contiguous elements of an operand (starting at element `off`) into shared
// memory as fp32, all threads of the CTA taking part.
__device__ __forceinline__ void load_to_smem(float* dst, const OperandDev& o, long long off, int cnt)
{
    for (int e = threadIdx.x; e < cnt; e += blockDim.x)
        dst[e] = load_elem(o, off + e);
}

// Output element `idx` of K / P / x / u: float32, or bfloat16 (round to nearest even) when the call asked for it.
// `base` is the caller's array whatever its element type; idx counts elements.
__device__ __forceinline__ void store_out(float* base, long long idx, float v, int bf16)
{
    if (bf16)
        reinterpret_cast<__nv_bfloat16*>(base)[idx] = __float2bfloat16_rn(v);
    else
        base[idx] = v;
}
// four consecutive elements starting at idx (idx a multiple of 4, base 16-byte aligned)
__device__ __forceinline__ void store_out4(float* base, long long idx, float4 v, int bf16)
{
    if (bf16) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
        uint2 w;
        w.x = *reinterpret_cast<uint32_t*>(&lo);
        w.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(base) + idx) = w;
    } else {
        *reinterpret_cast<float4*>(base + idx) = v;
    }
}

// Q = scale * U U' + diag(d) written out densely (float32, [N][n][n]) for the instances of the launch's token window:
// the state cost of the TTC layer is a combination of a few basis directions plus a diagonal (Parameterization
// paragraph), so a caller can hand over U [n][r] and d [n] instead of n x n numbers per instance.  One CTA per
// instance at a time; U', d staged in shared memory.
__global__ void __launch_bounds__(256) expand_lowrank_q_kernel(SolveParams p, OperandDev U, OperandDev d, int r, float scale,
                                                               float* Qdense)
{
    extern __shared__ float sm_u[];          // U' [r][n] then d [n]
    const int n = p.n;
    const long long nwin = p.b0 * p.b1 * p.tcount;
    for (long long w = blockIdx.x; w < nwin; w += gridDim.x) {
        const long long inst = window_instance(p, w);
        const long long ou = operand_offset(U, inst, p.b1, p.b2), od = operand_offset(d, inst, p.b1, p.b2);
        __syncthreads();
        for (int e = threadIdx.x; e < n * r; e += blockDim.x)
            sm_u[(e % r) * n + e / r] = load_elem(U, ou + e);
        for (int e = threadIdx.x; e < n; e += blockDim.x)
            sm_u[r * n + e] = load_elem(d, od + e);
        __syncthreads();
        float* dst = Qdense + inst * (long long)n * n;
        for (int e = threadIdx.x; e < n * n; e += blockDim.x) {
            const int i = e / n, j = e % n;
            float acc = 0.f;
            for (int k = 0; k < r; ++k)
                acc = fmaf(sm_u[k * n + i], sm_u[k * n + j], acc);
            acc *= scale;
            if (i == j)
                acc += sm_u[r * n + i];
            dst[e] = acc;
        }
    }
}

__device__ __forceinline__ float quiet_nan() { return __int_as_float(0x7fc00000); }

} // namespace ttc
