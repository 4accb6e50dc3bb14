// Riccati-backward kernel for n = m = 64 with tensor-core contractions (tf32 operands rounded
// to nearest, fp32 accumulate) and a blocked fp32-grade factorisation of S = R + B'P B.
//
// One persistent CTA per SM, 384 threads = 3 groups of 4 warps.  The CTA keeps the per-head
// operands A', B' (tf32) and R (fp32) in shared memory; each group owns one instance at a time and
// runs its horizon loop independently (named barriers per group), so that the tensor-pipe phases
// of one group overlap the latency-bound factorisation of another.
//
// Per step (Prop. 3.1), for the group's instance, with warp w owning rows 16w..16w+15:
//   V = P B, T = P A           mma; P is chained from the accumulator registers of the last step
//   S = R + B'V                mma -> shared (fp32)
//   Y = B'T,  Pn = Q + A'T     mma (Pn stays in registers)
//   Linv = chol(S)^{-1}        2 x 2 blocks of 32: one warp factors and inverts a diagonal block in
//                              registers (one row / column per lane); the off-diagonal block, the Schur
//                              complement and Linv21 are small 3 x tf32 (error-compensated) products
//   Z = Linv Y, Pn -= Z'Z      mma          (P_t = Q + A'P A - Y'S^{-1}Y)
//   K_t = -Linv' Z             mma, only when every K_t is wanted
//   u_0 = -Linv'(Linv (Y x_0)) fp32 mat-vec products, when only u_0 is wanted
// Shared-memory operands of a contraction are stored with the contraction index contiguous
// (row stride 72 floats): every fragment is one conflict-free 64-bit load.  Inside each 8-wide
// k-tile the mma k-slots (t, t+4) are mapped to columns (2t, 2t+1), which is also the layout of
// an accumulator tile, so accumulators feed the next contraction without a shuffle.
//
// Work distribution: chunks of 24 consecutive tokens of one (sequence, head) are handed out by a
// global atomic counter; the three groups take every third token of the chunk.
#pragma once

#include "common.cuh"

namespace ttc {
namespace mma64 {

constexpr int N = 64;            // n = m = 64
constexpr int LDK = 72;          // row stride of contraction-contiguous tf32 operands / fragment-layout fp32
constexpr int GROUPS = 3;
constexpr int GTHREADS = 128;
constexpr int THREADS = GROUPS * GTHREADS;
constexpr int CHUNK = 24;        // tokens per work item

struct Smem {
    float At[N * LDK];           // At[j][k] = tf32(A[k][j])
    float Bt[N * LDK];           // Bt[j][k] = tf32(B[k][j])
    float R[N * LDK];            // fp32, fragment-layout reads
    struct Group {
        float bufA[N * LDK];     // V', T', Y', Z' (tf32, transposed: contraction index contiguous)
        float bufS[N * LDK];     // S (fp32 row-major) -> Linv' blocks (11', 21', 22') and W' during the factorisation
        float Linv[N * LDK];     // fp32 row-major inverse Cholesky factor; block (0,1) is scratch
        float x[2 * N];          // x_t, u_t
        float red[2 * N];        // partial sums of mat-vec products
        float y0[N];             // Y x_0
        int flag;                // first failed pivot of this instance (0 = none)
        int pad[3];
    } g[GROUPS];
    int chunk;                   // current work item (broadcast)
};

__device__ __forceinline__ uint32_t to_tf32(float x)
{
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float round_tf32(float x) { return __uint_as_float(to_tf32(x)); }

__device__ __forceinline__ void mma_16x8x8(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                           uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                 "{%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void group_barrier(int gid)
{
    asm volatile("bar.sync %0, %1;" ::"r"(gid + 1), "r"(GTHREADS) : "memory");
}

// acc[nt][.] += Arows(16 x 64) * Bop, with the A rows read from shared memory (row stride LDK,
// contraction index contiguous; `Arow0` points at the tile's first row) and Bop[n][k] likewise.
// NEG negates the A operand.
template <bool NEG>
__device__ __forceinline__ void mma_smemA(float (&acc)[8][4], const float* __restrict__ Arow0,
                                          const float* __restrict__ Bop, int g, int t)
{
#pragma unroll
    for (int kt = 0; kt < 8; ++kt) {
        float2 lo = *reinterpret_cast<const float2*>(Arow0 + g * LDK + 8 * kt + 2 * t);
        float2 hi = *reinterpret_cast<const float2*>(Arow0 + (g + 8) * LDK + 8 * kt + 2 * t);
        if (NEG) {
            lo.x = -lo.x; lo.y = -lo.y; hi.x = -hi.x; hi.y = -hi.y;
        }
        const uint32_t a0 = __float_as_uint(lo.x), a2 = __float_as_uint(lo.y);
        const uint32_t a1 = __float_as_uint(hi.x), a3 = __float_as_uint(hi.y);
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float2 b = *reinterpret_cast<const float2*>(Bop + (8 * nt + g) * LDK + 8 * kt + 2 * t);
            mma_16x8x8(acc[nt], a0, a1, a2, a3, __float_as_uint(b.x), __float_as_uint(b.y));
        }
    }
}

// Same with the A rows taken from an accumulator-layout register tile (already tf32-rounded).
__device__ __forceinline__ void mma_regA(float (&acc)[8][4], const float (&a)[8][4],
                                         const float* __restrict__ Bop, int g, int t)
{
#pragma unroll
    for (int kt = 0; kt < 8; ++kt) {
        const uint32_t a0 = __float_as_uint(a[kt][0]), a2 = __float_as_uint(a[kt][1]);
        const uint32_t a1 = __float_as_uint(a[kt][2]), a3 = __float_as_uint(a[kt][3]);
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float2 b = *reinterpret_cast<const float2*>(Bop + (8 * nt + g) * LDK + 8 * kt + 2 * t);
            mma_16x8x8(acc[nt], a0, a1, a2, a3, __float_as_uint(b.x), __float_as_uint(b.y));
        }
    }
}

__device__ __forceinline__ void zero_acc(float (&acc)[8][4])
{
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e)
            acc[nt][e] = 0.f;
}

// accumulator tile (rows r0+g, r0+g+8) -> dst[col][row] (transposed, stride LDK), tf32-rounded
__device__ __forceinline__ void store_transposed_tf32(float* dst, const float (&acc)[8][4], int r0, int g, int t)
{
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        const int c = 8 * nt + 2 * t;
        dst[c * LDK + r0 + g] = round_tf32(acc[nt][0]);
        dst[(c + 1) * LDK + r0 + g] = round_tf32(acc[nt][1]);
        dst[c * LDK + r0 + g + 8] = round_tf32(acc[nt][2]);
        dst[(c + 1) * LDK + r0 + g + 8] = round_tf32(acc[nt][3]);
    }
}

// accumulator tile -> dst[row][col] (row-major fp32, stride ld)
__device__ __forceinline__ void store_rowmajor(float* dst, int ld, const float (&acc)[8][4], int r0, int g, int t)
{
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        const int c = 8 * nt + 2 * t;
        *reinterpret_cast<float2*>(dst + (r0 + g) * ld + c) = make_float2(acc[nt][0], acc[nt][1]);
        *reinterpret_cast<float2*>(dst + (r0 + g + 8) * ld + c) = make_float2(acc[nt][2], acc[nt][3]);
    }
}

__device__ __forceinline__ void load_fragment_layout(float (&acc)[8][4], const float* src, int ld, int r0, int g,
                                                     int t)
{
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        const int c = 8 * nt + 2 * t;
        const float2 lo = *reinterpret_cast<const float2*>(src + (r0 + g) * ld + c);
        const float2 hi = *reinterpret_cast<const float2*>(src + (r0 + g + 8) * ld + c);
        acc[nt][0] = lo.x; acc[nt][1] = lo.y; acc[nt][2] = hi.x; acc[nt][3] = hi.y;
    }
}

// ---- fp32-grade small products: 3 x tf32 (hi*hi + hi*lo + lo*hi), operands split on load ----------
__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo)
{
    hi = to_tf32(x);
    lo = to_tf32(x - __uint_as_float(hi));
}

// acc (16 x 16 tile: 2 n-tiles) += A(16 x 32) * B, A rows at `Arow0` (fp32, k contiguous, stride LDK),
// B given as Bop[n][k] (fp32, stride LDK) with n-tiles starting at row `n0` of Bop.
template <bool NEG>
__device__ __forceinline__ void mma3x_16x16x32(float (&acc)[2][4], const float* __restrict__ Arow0,
                                               const float* __restrict__ Bop, int g, int t)
{
#pragma unroll
    for (int kt = 0; kt < 4; ++kt) {
        float2 lo = *reinterpret_cast<const float2*>(Arow0 + g * LDK + 8 * kt + 2 * t);
        float2 hi = *reinterpret_cast<const float2*>(Arow0 + (g + 8) * LDK + 8 * kt + 2 * t);
        if (NEG) {
            lo.x = -lo.x; lo.y = -lo.y; hi.x = -hi.x; hi.y = -hi.y;
        }
        uint32_t ah[4], al[4];
        split_tf32(lo.x, ah[0], al[0]);
        split_tf32(hi.x, ah[1], al[1]);
        split_tf32(lo.y, ah[2], al[2]);
        split_tf32(hi.y, ah[3], al[3]);
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const float2 b = *reinterpret_cast<const float2*>(Bop + (8 * nt + g) * LDK + 8 * kt + 2 * t);
            uint32_t bh0, bl0, bh1, bl1;
            split_tf32(b.x, bh0, bl0);
            split_tf32(b.y, bh1, bl1);
            mma_16x8x8(acc[nt], al[0], al[1], al[2], al[3], bh0, bh1);
            mma_16x8x8(acc[nt], ah[0], ah[1], ah[2], ah[3], bl0, bl1);
            mma_16x8x8(acc[nt], ah[0], ah[1], ah[2], ah[3], bh0, bh1);
        }
    }
}

// ---- warp-level 32 x 32 Cholesky and triangular inverse (one row / one column per lane) -----------
// s[c] = row `lane` of an SPD block.  On return s holds row `lane` of L (entries above the diagonal are
// meaningless), rs = 1 / L[lane][lane].  Returns 0 or 1 + index of the first non-positive pivot.
__device__ __forceinline__ int warp_chol32(float (&s)[32], float& rs_own, int lane)
{
    int bad = 0;
    rs_own = 1.f;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        float d = __shfl_sync(0xffffffffu, s[j], j);
        if (!(d > 0.f)) {
            if (!bad)
                bad = j + 1;
            d = 1.f;
        }
        const float rs = rsqrtf(d);
        const float lij = s[j] * rs;
        s[j] = lij;
        if (lane == j)
            rs_own = rs;
#pragma unroll
        for (int c = j + 1; c < 32; ++c) {
            const float lc = __shfl_sync(0xffffffffu, lij, c);
            s[c] = fmaf(-lij, lc, s[c]);
        }
    }
    return bad;
}

// Lt: L' in shared memory (Lt[k][i] = L[i][k], stride LDK, fp32).  Lane c computes column c of L^{-1}:
// x[i] = Linv[i][c] (0 for i < c).
__device__ __forceinline__ void warp_trinv32(float (&x)[32], const float* __restrict__ Lt, float rs_own, int lane)
{
    float a[32];
#pragma unroll
    for (int i = 0; i < 32; ++i)
        a[i] = 0.f;
#pragma unroll
    for (int k = 0; k < 32; ++k) {
        const float rsk = __shfl_sync(0xffffffffu, rs_own, k);
        const float xk = (k == lane) ? rsk : ((k > lane) ? -a[k] * rsk : 0.f);
        x[k] = xk;
#pragma unroll
        for (int i4 = (k + 1) & ~3; i4 < 32; i4 += 4) {
            const float4 l4 = *reinterpret_cast<const float4*>(Lt + k * LDK + i4);
            if (i4 + 0 > k) a[i4 + 0] = fmaf(l4.x, xk, a[i4 + 0]);
            if (i4 + 1 > k) a[i4 + 1] = fmaf(l4.y, xk, a[i4 + 1]);
            if (i4 + 2 > k) a[i4 + 2] = fmaf(l4.z, xk, a[i4 + 2]);
            if (i4 + 3 > k) a[i4 + 3] = fmaf(l4.w, xk, a[i4 + 3]);
        }
    }
}

// One warp: factor the 32 x 32 SPD block at Sblk (row-major, stride LDK) and write its inverse
// Cholesky factor to LinvBlk (row-major) and, transposed, over Sblk itself.  Scratch: 32 x 32 (stride LDK).
__device__ __forceinline__ int warp_factor_block(float* Sblk, float* LinvBlk, float* scratch, int lane)
{
    float s[32];
#pragma unroll
    for (int c = 0; c < 32; c += 4) {
        const float4 v = *reinterpret_cast<const float4*>(Sblk + lane * LDK + c);
        s[c] = v.x; s[c + 1] = v.y; s[c + 2] = v.z; s[c + 3] = v.w;
    }
    float rs_own;
    const int bad = warp_chol32(s, rs_own, lane);
#pragma unroll
    for (int k = 0; k < 32; ++k)
        scratch[k * LDK + lane] = s[k];                 // Lt[k][i] = L[i][k]
    __syncwarp();
    float x[32];
    warp_trinv32(x, scratch, rs_own, lane);
#pragma unroll
    for (int i = 0; i < 32; ++i)
        LinvBlk[i * LDK + lane] = x[i];                 // Linv[i][c], c = lane
#pragma unroll
    for (int i = 0; i < 32; i += 4)
        *reinterpret_cast<float4*>(Sblk + lane * LDK + i) = make_float4(x[i], x[i + 1], x[i + 2], x[i + 3]);
    return bad;
}

// acc += A * Bop over k-tiles [kt0, kt1) with the A rows read from fp32 shared memory and rounded on load.
template <bool NEG>
__device__ __forceinline__ void mma_smemA_round(float (&acc)[8][4], const float* __restrict__ Arow0,
                                                const float* __restrict__ Bop, int g, int t, int kt0, int kt1)
{
#pragma unroll
    for (int kt = 0; kt < 8; ++kt) {
        if (kt < kt0 || kt >= kt1)
            continue;
        float2 lo = *reinterpret_cast<const float2*>(Arow0 + g * LDK + 8 * kt + 2 * t);
        float2 hi = *reinterpret_cast<const float2*>(Arow0 + (g + 8) * LDK + 8 * kt + 2 * t);
        if (NEG) {
            lo.x = -lo.x; lo.y = -lo.y; hi.x = -hi.x; hi.y = -hi.y;
        }
        const uint32_t a0 = to_tf32(lo.x), a2 = to_tf32(lo.y), a1 = to_tf32(hi.x), a3 = to_tf32(hi.y);
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float2 b = *reinterpret_cast<const float2*>(Bop + (8 * nt + g) * LDK + 8 * kt + 2 * t);
            mma_16x8x8(acc[nt], a0, a1, a2, a3, __float_as_uint(b.x), __float_as_uint(b.y));
        }
    }
}

// Q (global, fp32 or bf16, row-major 64 x 64 at element offset oq) -> accumulator layout
__device__ __forceinline__ void load_Q_fragment(float (&acc)[8][4], const OperandDev& Q, long long oq, int r0, int g,
                                                int t)
{
    if (Q.dtype == TTC_BF16) {
        const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(Q.ptr) + oq;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const int c = 8 * nt + 2 * t;
            const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(q + (r0 + g) * N + c));
            const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(q + (r0 + g + 8) * N + c));
            acc[nt][0] = lo.x; acc[nt][1] = lo.y; acc[nt][2] = hi.x; acc[nt][3] = hi.y;
        }
    } else {
        const float* q = reinterpret_cast<const float*>(Q.ptr) + oq;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const int c = 8 * nt + 2 * t;
            const float2 lo = *reinterpret_cast<const float2*>(q + (r0 + g) * N + c);
            const float2 hi = *reinterpret_cast<const float2*>(q + (r0 + g + 8) * N + c);
            acc[nt][0] = lo.x; acc[nt][1] = lo.y; acc[nt][2] = hi.x; acc[nt][3] = hi.y;
        }
    }
}

__device__ __forceinline__ void group_fail_instance(const SolveParams& p, long long inst, int code, int gt)
{
    const int H = p.H;
    const float qn = quiet_nan();
    if (p.K)
        for (long long e = gt; e < (long long)H * N * N; e += GTHREADS)
            p.K[inst * (long long)H * N * N + e] = qn;
    if (p.P) {
        const long long cnt = (long long)(p.first_only ? 1 : H + 1) * N * N;
        for (long long e = gt; e < cnt; e += GTHREADS)
            p.P[inst * cnt + e] = qn;
    }
    if (p.x)
        for (long long e = gt; e < (long long)(H + 1) * N; e += GTHREADS)
            p.x[inst * (long long)(H + 1) * N + e] = qn;
    if (p.u) {
        const long long cnt = p.first_only ? N : (long long)H * N;
        for (long long e = gt; e < cnt; e += GTHREADS)
            p.u[inst * cnt + e] = qn;
    }
    if (p.info && gt == 0)
        p.info[inst] = code;
}


// Blocked factorisation of the group's S (fp32 row-major in bufS): on return G.Linv holds
// Linv = chol(S)^{-1} (row-major, lower triangle; block (0,1) is scratch) and bufS holds the blocks of
// Linv' (11' at (0,0), 22' at (1,1), 21' at (0,1) when `want_transposed`; block (1,0) is scratch).
// All 128 threads of the group call it.  A non-positive pivot is recorded in G.flag as `code0` + index.
__device__ __forceinline__ void group_factor_invert(Smem::Group& G, int gid, int w, int lane, int g, int t,
                                                    bool want_transposed, int code0)
{
    const int mt = w >> 1, nh = w & 1;          // 16 x 16 tile of a 32 x 32 block owned by this warp
    float* S = G.bufS;
    float* Li = G.Linv;
    if (w == 0) {
        const int bad = warp_factor_block(S, Li, Li + 32, lane);
        if (bad && lane == 0 && G.flag == 0)
            G.flag = code0 + bad;
    }
    group_barrier(gid);
    float acc[2][4];
    // L21 = S21 Linv11'  -> Linv block (1,0) (temporarily)
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e)
            acc[nt][e] = 0.f;
    mma3x_16x16x32<false>(acc, S + (32 + 16 * mt) * LDK, Li + (16 * nh) * LDK, g, t);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        const int c = 16 * nh + 8 * nt + 2 * t;
        *reinterpret_cast<float2*>(Li + (32 + 16 * mt + g) * LDK + c) = make_float2(acc[nt][0], acc[nt][1]);
        *reinterpret_cast<float2*>(Li + (32 + 16 * mt + g + 8) * LDK + c) = make_float2(acc[nt][2], acc[nt][3]);
    }
    group_barrier(gid);
    // S22 -= L21 L21'  (in place)
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        const int c = 32 + 16 * nh + 8 * nt + 2 * t;
        const float2 lo = *reinterpret_cast<const float2*>(S + (32 + 16 * mt + g) * LDK + c);
        const float2 hi = *reinterpret_cast<const float2*>(S + (32 + 16 * mt + g + 8) * LDK + c);
        acc[nt][0] = lo.x; acc[nt][1] = lo.y; acc[nt][2] = hi.x; acc[nt][3] = hi.y;
    }
    mma3x_16x16x32<true>(acc, Li + (32 + 16 * mt) * LDK, Li + (32 + 16 * nh) * LDK, g, t);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        const int c = 32 + 16 * nh + 8 * nt + 2 * t;
        *reinterpret_cast<float2*>(S + (32 + 16 * mt + g) * LDK + c) = make_float2(acc[nt][0], acc[nt][1]);
        *reinterpret_cast<float2*>(S + (32 + 16 * mt + g + 8) * LDK + c) = make_float2(acc[nt][2], acc[nt][3]);
    }
    // W = L21 Linv11 -> W' in bufS block (1,0)   (Linv11' sits in bufS block (0,0))
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e)
            acc[nt][e] = 0.f;
    mma3x_16x16x32<false>(acc, Li + (32 + 16 * mt) * LDK, S + (16 * nh) * LDK, g, t);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        const int c = 16 * nh + 8 * nt + 2 * t;
        const int r = 16 * mt + g;
        S[(32 + c) * LDK + r] = acc[nt][0];
        S[(32 + c + 1) * LDK + r] = acc[nt][1];
        S[(32 + c) * LDK + r + 8] = acc[nt][2];
        S[(32 + c + 1) * LDK + r + 8] = acc[nt][3];
    }
    group_barrier(gid);
    if (w == 0) {
        const int bad = warp_factor_block(S + 32 * LDK + 32, Li + 32 * LDK + 32, Li + 32, lane);
        if (bad && lane == 0 && G.flag == 0)
            G.flag = code0 + 32 + bad;
    }
    group_barrier(gid);
    // Linv21 = -Linv22 W
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e)
            acc[nt][e] = 0.f;
    mma3x_16x16x32<true>(acc, Li + (32 + 16 * mt) * LDK + 32, S + (32 + 16 * nh) * LDK, g, t);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        const int c = 16 * nh + 8 * nt + 2 * t;
        *reinterpret_cast<float2*>(Li + (32 + 16 * mt + g) * LDK + c) = make_float2(acc[nt][0], acc[nt][1]);
        *reinterpret_cast<float2*>(Li + (32 + 16 * mt + g + 8) * LDK + c) = make_float2(acc[nt][2], acc[nt][3]);
        if (want_transposed) {
            const int r = 32 + 16 * mt + g;
            S[c * LDK + r] = acc[nt][0];
            S[(c + 1) * LDK + r] = acc[nt][1];
            S[c * LDK + r + 8] = acc[nt][2];
            S[(c + 1) * LDK + r + 8] = acc[nt][3];
        }
    }
    group_barrier(gid);
}

__global__ void __launch_bounds__(THREADS, 1) riccati_mma64_kernel(SolveParams p, int* chunk_counter)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
    const int tid = threadIdx.x;
    const int gid = tid / GTHREADS;          // group
    const int gt = tid % GTHREADS;           // thread in group
    const int w = gt >> 5;                   // warp in group: rows 16w..16w+15 of every product
    const int lane = gt & 31;
    const int g = lane >> 2, t = lane & 3;   // mma fragment coordinates
    const int i = gt & 63, h = gt >> 6;      // mat-vec layout of the rollout: row i, column half h
    const int r0 = 16 * w;
    Smem::Group& G = sm.g[gid];
    const int H = p.H;
    const long long chunks_per_head = (p.b2 + CHUNK - 1) / CHUNK;
    const long long nchunks = p.b0 * p.b1 * chunks_per_head;
    const bool need_K_all = (p.K != nullptr) || (p.x != nullptr) || (p.u != nullptr && !p.first_only);
    const bool want_u0 = (p.u != nullptr) && p.first_only;
    float* Kbase = p.K ? p.K : p.Kws;
    long long offA_loaded = -1, offB_loaded = -1, offR_loaded = -1;

    for (;;) {
        __syncthreads();
        if (tid == 0)
            sm.chunk = atomicAdd(chunk_counter, 1);
        __syncthreads();
        const long long chunk = sm.chunk;
        if (chunk >= nchunks)
            break;
        const long long head = chunk / chunks_per_head;            // (sequence, head) pair index
        const long long tok0 = (chunk % chunks_per_head) * CHUNK;
        const long long inst0 = head * p.b2 + tok0;
        const int ntok = (int)min((long long)CHUNK, p.b2 - tok0);
        {
            const long long oa = operand_offset(p.A, inst0, p.b1, p.b2);
            const long long ob = operand_offset(p.B, inst0, p.b1, p.b2);
            const long long orr = operand_offset(p.R, inst0, p.b1, p.b2);
            if (oa != offA_loaded || ob != offB_loaded || orr != offR_loaded) {
                const float* Ag = reinterpret_cast<const float*>(p.A.ptr) + oa;
                const float* Bg = reinterpret_cast<const float*>(p.B.ptr) + ob;
                const float* Rg = reinterpret_cast<const float*>(p.R.ptr) + orr;
                for (int e = tid; e < N * N; e += THREADS) {
                    const int k = e >> 6, j = e & 63;
                    sm.At[j * LDK + k] = round_tf32(Ag[e]);
                    sm.Bt[j * LDK + k] = round_tf32(Bg[e]);
                    sm.R[k * LDK + j] = Rg[e];
                }
                offA_loaded = oa; offB_loaded = ob; offR_loaded = orr;
                __syncthreads();
            }
        }

        for (int tk = gid; tk < ntok; tk += GROUPS) {
            const long long inst = inst0 + tk;
            const long long oq = operand_offset(p.Q, inst, p.b1, p.b2);
            if (p.x0.ptr && gt < N)
                G.x[gt] = load_elem(p.x0, operand_offset(p.x0, inst, p.b1, p.b2) + gt);
            if (gt == 0)
                G.flag = 0;
            float P[8][4];                       // value matrix rows r0+g, r0+g+8 (fp32, then tf32 in place)
            load_Q_fragment(P, p.Q, oq, r0, g, t);              // P_H = Q
            float* Pout = p.P ? p.P + inst * (long long)(p.first_only ? 1 : H + 1) * N * N : nullptr;
            if (Pout && !p.first_only)
                store_rowmajor(Pout + (long long)H * N * N, N, P, r0, g, t);
            float* Kout = Kbase ? Kbase + inst * (long long)H * N * N : nullptr;
            group_barrier(gid);

            for (int ts = H - 1; ts >= 0; --ts) {
#pragma unroll
                for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        P[nt][e] = round_tf32(P[nt][e]);
                float acc[8][4];
                // V = P B  -> V' (tf32) in bufA
                zero_acc(acc);
                mma_regA(acc, P, sm.Bt, g, t);
                store_transposed_tf32(G.bufA, acc, r0, g, t);
                // T = P A (kept in registers until V' has been consumed)
                float T[8][4];
                zero_acc(T);
                mma_regA(T, P, sm.At, g, t);
                load_Q_fragment(P, p.Q, oq, r0, g, t);          // accumulator of P_t starts at Q
                group_barrier(gid);
                // S = R + B'V -> bufS (fp32 row-major)
                load_fragment_layout(acc, sm.R, LDK, r0, g, t);
                mma_smemA<false>(acc, sm.Bt + r0 * LDK, G.bufA, g, t);
                store_rowmajor(G.bufS, LDK, acc, r0, g, t);
                group_barrier(gid);
                store_transposed_tf32(G.bufA, T, r0, g, t);     // T'
                group_barrier(gid);
                // Y = B'T ; Pn = Q + A'T
                zero_acc(acc);
                mma_smemA<false>(acc, sm.Bt + r0 * LDK, G.bufA, g, t);
                mma_smemA<false>(P, sm.At + r0 * LDK, G.bufA, g, t);
                if (ts == 0 && want_u0) {                       // y0 = Y x_0 (fp32)
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) {
                        const float xa = G.x[8 * nt + 2 * t], xb = G.x[8 * nt + 2 * t + 1];
                        s0 = fmaf(acc[nt][0], xa, fmaf(acc[nt][1], xb, s0));
                        s1 = fmaf(acc[nt][2], xa, fmaf(acc[nt][3], xb, s1));
                    }
                    s0 += __shfl_xor_sync(0xffffffffu, s0, 1);
                    s0 += __shfl_xor_sync(0xffffffffu, s0, 2);
                    s1 += __shfl_xor_sync(0xffffffffu, s1, 1);
                    s1 += __shfl_xor_sync(0xffffffffu, s1, 2);
                    if (t == 0) {
                        G.y0[r0 + g] = s0;
                        G.y0[r0 + g + 8] = s1;
                    }
                }
                group_barrier(gid);                             // T' consumed
                store_transposed_tf32(G.bufA, acc, r0, g, t);   // Y'
                // ---- Linv = chol(S)^{-1}
                group_factor_invert(G, gid, w, lane, g, t, need_K_all, ts * N);
                // Z = Linv Y  (Linv lower triangular: rows < 32 only need k < 32)
                zero_acc(acc);
                mma_smemA_round<false>(acc, G.Linv + r0 * LDK, G.bufA, g, t, 0, (w < 2) ? 4 : 8);
                group_barrier(gid);                             // Y' consumed
                store_transposed_tf32(G.bufA, acc, r0, g, t);   // Z'
                group_barrier(gid);
                // Pn -= Z'Z
                mma_smemA<true>(P, G.bufA + r0 * LDK, G.bufA, g, t);
                if (need_K_all) {                               // K_t = -Linv' Z
                    zero_acc(acc);
                    mma_smemA_round<true>(acc, G.bufS + r0 * LDK, G.bufA, g, t, (w < 2) ? 0 : 4, 8);
                    store_rowmajor(Kout + (long long)ts * N * N, N, acc, r0, g, t);
                }
                if (Pout && (!p.first_only || ts == 0))
                    store_rowmajor(Pout + (long long)(p.first_only ? 0 : ts) * N * N, N, P, r0, g, t);
                group_barrier(gid);      // Z', Linv' consumed before the next step overwrites them
            }

            const int fail = G.flag;         // written before the barriers above
            if (fail) {
                group_barrier(gid);
                group_fail_instance(p, inst, fail, gt);
                group_barrier(gid);
                continue;
            }
            if (p.info && gt == 0)
                p.info[inst] = 0;
            if (want_u0) {                   // u_0 = -Linv' (Linv y0), fp32
                if (gt < N) {
                    float v = 0.f;
                    for (int k = 0; k <= gt; ++k)
                        v = fmaf(G.Linv[gt * LDK + k], G.y0[k], v);
                    G.red[gt] = v;
                }
                group_barrier(gid);
                if (gt < N) {
                    float v = 0.f;
                    for (int k = gt; k < N; ++k)
                        v = fmaf(G.Linv[k * LDK + gt], G.red[k], v);
                    p.u[inst * (long long)N + gt] = -v;
                }
            }
            // ---- forward rollout (Alg. 1): u_t = K_t x_t, x_{t+1} = A x_t + B u_t, fp32, from global K_t
            if (p.x || (p.u && !p.first_only)) {
                const float* Ag = reinterpret_cast<const float*>(p.A.ptr) + offA_loaded;
                const float* Bg = reinterpret_cast<const float*>(p.B.ptr) + offB_loaded;
                float* xo = p.x ? p.x + inst * (long long)(H + 1) * N : nullptr;
                float* uo = (p.u && !p.first_only) ? p.u + inst * (long long)H * N : nullptr;
                __threadfence_block();
                group_barrier(gid);
                if (xo && gt < N)
                    xo[gt] = G.x[gt];
                for (int ts = 0; ts < H; ++ts) {
                    const float* Kt = Kout + (long long)ts * N * N + i * N + 32 * h;
                    float part = 0.f;
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        const float4 kv = *reinterpret_cast<const float4*>(Kt + c);
                        part = fmaf(kv.x, G.x[32 * h + c], part);
                        part = fmaf(kv.y, G.x[32 * h + c + 1], part);
                        part = fmaf(kv.z, G.x[32 * h + c + 2], part);
                        part = fmaf(kv.w, G.x[32 * h + c + 3], part);
                    }
                    G.red[64 * h + i] = part;
                    group_barrier(gid);
                    if (gt < N) {
                        const float uv = G.red[gt] + G.red[64 + gt];
                        G.x[N + gt] = uv;                         // u_t
                        if (uo)
                            uo[(long long)ts * N + gt] = uv;
                    }
                    group_barrier(gid);
                    float part2 = 0.f;
                    const float* Ar = Ag + i * N + 32 * h;
                    const float* Br = Bg + i * N + 32 * h;
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        const float4 av = *reinterpret_cast<const float4*>(Ar + c);
                        const float4 bv = *reinterpret_cast<const float4*>(Br + c);
                        part2 = fmaf(av.x, G.x[32 * h + c], part2);
                        part2 = fmaf(av.y, G.x[32 * h + c + 1], part2);
                        part2 = fmaf(av.z, G.x[32 * h + c + 2], part2);
                        part2 = fmaf(av.w, G.x[32 * h + c + 3], part2);
                        part2 = fmaf(bv.x, G.x[N + 32 * h + c], part2);
                        part2 = fmaf(bv.y, G.x[N + 32 * h + c + 1], part2);
                        part2 = fmaf(bv.z, G.x[N + 32 * h + c + 2], part2);
                        part2 = fmaf(bv.w, G.x[N + 32 * h + c + 3], part2);
                    }
                    G.red[64 * h + i] = part2;
                    group_barrier(gid);
                    if (gt < N) {
                        const float xv = G.red[gt] + G.red[64 + gt];
                        G.x[gt] = xv;
                        if (xo)
                            xo[(long long)(ts + 1) * N + gt] = xv;
                    }
                    group_barrier(gid);
                }
            }
            group_barrier(gid);
        }
    }
}

inline size_t smem_bytes() { return sizeof(Smem); }

} // namespace mma64
} // namespace ttc
