// Riccati-backward kernel for n = m = 64 with tensor-core contractions (tf32 operands rounded
// to nearest, fp32 accumulate) and an fp32 in-register factorisation.
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
//   [S | Y] -> registers, one half row per thread; 64-step elimination: S = L L', Z = L^{-1} Y
//   Pn -= Z'Z                  mma          (P_t = Q + A'P A - Y'S^{-1}Y)
//   K_t = -L^{-T} Z            64-step back substitution, only when K_t is needed
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
constexpr int LDR = 68;          // row stride of row-major fp32 matrices read one half row per thread
constexpr int GROUPS = 3;
constexpr int GTHREADS = 128;
constexpr int THREADS = GROUPS * GTHREADS;
constexpr int CHUNK = 24;        // tokens per work item

struct Smem {
    float At[N * LDK];           // At[j][k] = tf32(A[k][j])
    float Bt[N * LDK];           // Bt[j][k] = tf32(B[k][j])
    float R[N * LDK];            // fp32, fragment-layout reads
    struct Group {
        float bufA[N * LDK];     // V', T' (tf32) -> Y (fp32 row-major, LDR) -> Z' (tf32)
        float bufS[N * LDR];     // S (fp32 row-major, LDR) -> exchange buffers of the eliminations
        float Q[N * LDK];        // fp32
        float x[2 * N];          // x_t, scratch
        float red[2 * N];        // partial sums of mat-vec products
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

__device__ __forceinline__ float select4x8(const float (&v)[32], int q, int jj)
{
    // v[8*q + jj] with jj a compile-time constant after unrolling and q in 0..3 at run time
    float r = v[jj];
    r = (q == 1) ? v[8 + jj] : r;
    r = (q == 2) ? v[16 + jj] : r;
    r = (q == 3) ? v[24 + jj] : r;
    return r;
}
__device__ __forceinline__ void assign4x8(float (&v)[32], int q, int jj, float x)
{
    v[jj] = (q == 0) ? x : v[jj];
    v[8 + jj] = (q == 1) ? x : v[8 + jj];
    v[16 + jj] = (q == 2) ? x : v[16 + jj];
    v[24 + jj] = (q == 3) ? x : v[24 + jj];
}

// Elimination on [S | Y] held one half row per thread (thread (i, h): columns 32h..32h+31 of row i):
// on return s holds the rows of L (S = L L'), y the rows of Z = L^{-1} Y, rs = 1 / L[i][i].
// xch: 2 x (64 + 64) floats of exchange space.  Returns 0 or 1 + index of the first non-positive pivot.
__device__ __forceinline__ int eliminate_forward(float (&s)[32], float (&y)[32], float& rs_own, float* xch,
                                                 int i, int h, int gid)
{
    int bad = 0;
    rs_own = 0.f;
#pragma unroll 1
    for (int jo = 0; jo < 8; ++jo) {
        const int hj = jo >> 2, q = jo & 3;
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
            const int j = 8 * jo + jj;
            float* col = xch + (j & 1) * 128;
            float* zr = col + 64;
            if (h == hj) {
                const float v = select4x8(s, q, jj);
                col[i] = (i >= j) ? v : 0.f;
            }
            if (i == j) {
#pragma unroll
                for (int c = 0; c < 32; c += 4)
                    *reinterpret_cast<float4*>(zr + 32 * h + c) = make_float4(y[c], y[c + 1], y[c + 2], y[c + 3]);
            }
            group_barrier(gid);
            float d = col[j];
            if (!(d > 0.f)) {
                if (!bad)
                    bad = j + 1;
                d = 1.f;
            }
            const float rs = rsqrtf(d);
            const float ci = col[i];
            const float f = (i > j) ? ci * (rs * rs) : 0.f;
            if (i == j)
                rs_own = rs;
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
                const float4 cv = *reinterpret_cast<const float4*>(col + 32 * h + c);
                s[c] = fmaf(-f, cv.x, s[c]);
                s[c + 1] = fmaf(-f, cv.y, s[c + 1]);
                s[c + 2] = fmaf(-f, cv.z, s[c + 2]);
                s[c + 3] = fmaf(-f, cv.w, s[c + 3]);
            }
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
                const float4 zv = *reinterpret_cast<const float4*>(zr + 32 * h + c);
                y[c] = fmaf(-f, zv.x, y[c]);
                y[c + 1] = fmaf(-f, zv.y, y[c + 1]);
                y[c + 2] = fmaf(-f, zv.z, y[c + 2]);
                y[c + 3] = fmaf(-f, zv.w, y[c + 3]);
            }
            if (h == hj)
                assign4x8(s, q, jj, ci * rs);      // L[i][j] (0 above the diagonal)
        }
    }
#pragma unroll
    for (int c = 0; c < 32; ++c)
        y[c] *= rs_own;
    return bad;
}

// Back substitution: z (rows of Z) <- rows of L^{-T} Z, with l the rows of L.
__device__ __forceinline__ void eliminate_backward(float (&z)[32], const float (&l)[32], float rs_own, float* xch,
                                                   int i, int h, int gid)
{
#pragma unroll 2
    for (int r = N - 1; r >= 0; --r) {
        float* kr = xch + (r & 1) * 128;
        float* lr = kr + 64;
        if (i == r) {
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
                z[c] *= rs_own; z[c + 1] *= rs_own; z[c + 2] *= rs_own; z[c + 3] *= rs_own;
                *reinterpret_cast<float4*>(kr + 32 * h + c) = make_float4(z[c], z[c + 1], z[c + 2], z[c + 3]);
                *reinterpret_cast<float4*>(lr + 32 * h + c) = make_float4(l[c], l[c + 1], l[c + 2], l[c + 3]);
            }
        }
        group_barrier(gid);
        const float f = (i < r) ? lr[i] : 0.f;
#pragma unroll
        for (int c = 0; c < 32; c += 4) {
            const float4 kv = *reinterpret_cast<const float4*>(kr + 32 * h + c);
            z[c] = fmaf(-f, kv.x, z[c]);
            z[c + 1] = fmaf(-f, kv.y, z[c + 1]);
            z[c + 2] = fmaf(-f, kv.z, z[c + 2]);
            z[c + 3] = fmaf(-f, kv.w, z[c + 3]);
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
    const int i = gt & 63, h = gt >> 6;      // elimination layout: row i, column half h
    const int r0 = 16 * w;
    Smem::Group& G = sm.g[gid];
    const int H = p.H;
    const long long chunks_per_head = (p.b2 + CHUNK - 1) / CHUNK;
    const long long nchunks = p.b0 * p.b1 * chunks_per_head;
    const bool need_K_all = (p.K != nullptr) || (p.x != nullptr) || (p.u != nullptr && !p.first_only);
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
            // ---- load Q (fp32 in shared memory, fragment layout reads), x0
            {
                const long long oq = operand_offset(p.Q, inst, p.b1, p.b2);
                if (p.Q.dtype == TTC_BF16) {
                    const __nv_bfloat162* q2 = reinterpret_cast<const __nv_bfloat162*>(
                        reinterpret_cast<const __nv_bfloat16*>(p.Q.ptr) + oq);
                    for (int e = gt; e < N * N / 2; e += GTHREADS) {
                        const float2 v = __bfloat1622float2(q2[e]);
                        const int r = (2 * e) >> 6, c = (2 * e) & 63;
                        *reinterpret_cast<float2*>(G.Q + r * LDK + c) = v;
                    }
                } else {
                    const float4* q4 = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.Q.ptr) + oq);
                    for (int e = gt; e < N * N / 4; e += GTHREADS) {
                        const float4 v = q4[e];
                        const int r = (4 * e) >> 6, c = (4 * e) & 63;
                        *reinterpret_cast<float4*>(G.Q + r * LDK + c) = v;
                    }
                }
                if (p.x0.ptr && gt < N)
                    G.x[gt] = load_elem(p.x0, operand_offset(p.x0, inst, p.b1, p.b2) + gt);
            }
            group_barrier(gid);

            float P[8][4];                       // value matrix rows r0+g, r0+g+8 (fp32, then tf32 in place)
            load_fragment_layout(P, G.Q, LDK, r0, g, t);        // P_H = Q
            float* Pout = p.P ? p.P + inst * (long long)(p.first_only ? 1 : H + 1) * N * N : nullptr;
            if (Pout && !p.first_only)
                store_rowmajor(Pout + (long long)H * N * N, N, P, r0, g, t);
            float* Kout = Kbase ? Kbase + inst * (long long)H * N * N : nullptr;
            int fail = 0;

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
                group_barrier(gid);
                // S = R + B'V -> bufS (fp32 row-major)
                load_fragment_layout(acc, sm.R, LDK, r0, g, t);
                mma_smemA<false>(acc, sm.Bt + r0 * LDK, G.bufA, g, t);
                store_rowmajor(G.bufS, LDR, acc, r0, g, t);
                group_barrier(gid);
                store_transposed_tf32(G.bufA, T, r0, g, t);     // T'
                group_barrier(gid);
                // Y = B'T ; Pn = Q + A'T
                zero_acc(acc);
                mma_smemA<false>(acc, sm.Bt + r0 * LDK, G.bufA, g, t);
                load_fragment_layout(P, G.Q, LDK, r0, g, t);
                mma_smemA<false>(P, sm.At + r0 * LDK, G.bufA, g, t);
                group_barrier(gid);
                store_rowmajor(G.bufA, LDR, acc, r0, g, t);     // Y (fp32 row-major)
                group_barrier(gid);
                // ---- elimination on [S | Y], one half row per thread
                float s[32], y[32];
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    const float4 sv = *reinterpret_cast<const float4*>(G.bufS + i * LDR + 32 * h + c);
                    const float4 yv = *reinterpret_cast<const float4*>(G.bufA + i * LDR + 32 * h + c);
                    s[c] = sv.x; s[c + 1] = sv.y; s[c + 2] = sv.z; s[c + 3] = sv.w;
                    y[c] = yv.x; y[c + 1] = yv.y; y[c + 2] = yv.z; y[c + 3] = yv.w;
                }
                group_barrier(gid);
                float rs_own;
                const int bad = eliminate_forward(s, y, rs_own, G.bufS, i, h, gid);
                if (bad && !fail)
                    fail = ts * N + bad;
                // Z' (tf32) -> bufA
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    G.bufA[(32 * h + c) * LDK + i] = round_tf32(y[c]);
                group_barrier(gid);
                // Pn -= Z'Z
                mma_smemA<true>(P, G.bufA + r0 * LDK, G.bufA, g, t);
                const bool needK = need_K_all || ts == 0;
                if (needK) {
                    eliminate_backward(y, s, rs_own, G.bufS, i, h, gid);     // y <- rows of L^{-T} Z = -K_t
                    if (Kout && need_K_all) {
                        float* dst = Kout + (long long)ts * N * N + i * N + 32 * h;
#pragma unroll
                        for (int c = 0; c < 32; c += 4)
                            *reinterpret_cast<float4*>(dst + c) = make_float4(-y[c], -y[c + 1], -y[c + 2], -y[c + 3]);
                    }
                    if (ts == 0 && p.u && p.first_only) {                    // u_0 = K_0 x_0
                        float part = 0.f;
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            part = fmaf(-y[c], G.x[32 * h + c], part);
                        G.red[64 * h + i] = part;
                    }
                }
                if (Pout && (!p.first_only || ts == 0))
                    store_rowmajor(Pout + (long long)(p.first_only ? 0 : ts) * N * N, N, P, r0, g, t);
                group_barrier(gid);      // Z' consumed, exchange buffers idle, red[] complete
            }

            if (fail) {
                group_fail_instance(p, inst, fail, gt);
                group_barrier(gid);
                continue;
            }
            if (p.info && gt == 0)
                p.info[inst] = 0;
            if (p.u && p.first_only && gt < N)
                p.u[inst * (long long)N + gt] = G.red[gt] + G.red[64 + gt];
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
