// Measured FP32 FMA peak of the device: the denominator of every "bound: alu" roofline fraction.
// A register-resident FMA chain kernel (no memory traffic): every thread advances 8 independent accumulators, so
// that with 32 warps per SM the 4-cycle FMA latency is covered many times over.  Two variants: scalar fma.rn.f32
// and the packed fma.rn.f32x2 that the dense loops of the fp32 kernels use; the larger rate is the peak.
#pragma once

#include "common.cuh"

namespace ttc {
namespace probe {

constexpr int THREADS = 1024;
constexpr int CHAINS = 8;

template <bool PACKED>
__global__ void __launch_bounds__(THREADS, 1) fma_chain_kernel(int iters, float seed, float* sink)
{
    float acc[2 * CHAINS];
#pragma unroll
    for (int i = 0; i < 2 * CHAINS; ++i)
        acc[i] = seed + (float)(threadIdx.x + i);
    const float a = 1.0f - 1e-7f * seed, b = 1e-9f * seed;
    if (PACKED) {
        unsigned long long v[CHAINS], aa, bb;
        asm("mov.b64 %0, {%1, %2};" : "=l"(aa) : "f"(a), "f"(a));
        asm("mov.b64 %0, {%1, %2};" : "=l"(bb) : "f"(b), "f"(b));
#pragma unroll
        for (int i = 0; i < CHAINS; ++i)
            asm("mov.b64 %0, {%1, %2};" : "=l"(v[i]) : "f"(acc[2 * i]), "f"(acc[2 * i + 1]));
#pragma unroll 1
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int rep = 0; rep < 4; ++rep)
#pragma unroll
                for (int i = 0; i < CHAINS; ++i)
                    asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(v[i]) : "l"(aa), "l"(bb));
        }
#pragma unroll
        for (int i = 0; i < CHAINS; ++i)
            asm("mov.b64 {%0, %1}, %2;" : "=f"(acc[2 * i]), "=f"(acc[2 * i + 1]) : "l"(v[i]));
    } else {
#pragma unroll 1
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int rep = 0; rep < 4; ++rep)
#pragma unroll
                for (int i = 0; i < 2 * CHAINS; ++i)
                    asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(acc[i]) : "f"(a), "f"(b));
        }
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 2 * CHAINS; ++i)
        s += acc[i];
    if (s == 123.456f)                       // never true in practice: keeps the chains alive
        sink[threadIdx.x] = s;
}

// flops of one launch: every thread does iters * 4 * 2*CHAINS FMAs in both variants
inline double launch_flops(int blocks, int iters) { return 2.0 * (double)blocks * THREADS * iters * 4.0 * 2 * CHAINS; }

} // namespace probe
} // namespace ttc
