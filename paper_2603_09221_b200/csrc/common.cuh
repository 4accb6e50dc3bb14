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

__device__ __forceinline__ float quiet_nan() { return __int_as_float(0x7fc00000); }

} // namespace ttc
