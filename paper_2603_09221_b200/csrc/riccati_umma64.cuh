// Riccati-backward kernel for n = m = 64 on the 5th-generation tensor cores (tcgen05.mma,
// kind::tf32, fp32 accumulators in tensor memory).
//
// One persistent CTA per SM, 512 threads = 4 warpgroups.  A warpgroup (128 threads = the 128 lanes of tensor
// memory) walks ONE instance through the horizon; the four warpgroups are independent (own operands, own barriers,
// own quarter of tensor memory) and share the per-head operand BA = [B'; A'] (128 x 64).  The step is one long
// dependency chain (64 pivots in 8 panels); four chains per SM keep the tensor pipe, the shared-memory pipe and
// the issue slots busier than fewer, longer ones (a thread has 128 registers).
//
// Per step (Prop. 3.1), with P symmetric:
//   (1)  W  = BA * P                  -> W = [V'; T'] = [(P B)'; (P A)']                    SS, M128 N64
//   (2)  F  = W * B  = [S - R ; Y']                                                        TS (A operand read from
//        tensor memory, no round trip through shared memory), N64.  The issuing thread waits for (1) first: an MMA
//        that reads its A operand from tensor memory is not ordered after the MMAs that wrote it.
//   (3)  right-looking blocked Cholesky (8-wide panels) of the tall matrix G = [S; Y'] IN TENSOR MEMORY:
//        thread r owns row r (lane r).  Per panel: load the row's 8 panel columns (tcgen05.ld), add R, the warp that
//        owns the 8 diagonal rows factors the 8 x 8 block in registers and publishes it, every thread
//        forward-substitutes its own row, writes it as tf32 hi + lo parts to a 128 x 8 operand buffer, and ONE
//        rank-8 tcgen05.mma (3 passes: hi*hi + lo*hi + hi*lo, error-compensated) applies the trailing update to all
//        128 rows.  It leaves L (S = L L') and Z' = Y' L^{-T} (rows 64..127): no explicit inverse.
//   (4)  DP = W * A = [ . ; A'P A]   (into the columns that held F)                         TS, N64
//   (5)  DP -= Z' Z                                                                         SS, N64
//   P <- Q + DP                  (P_t = Q + A'P A - Y'S^{-1}Y)
//   Gains (every K_t wanted): rows 0..63 of the factorisation keep going after their diagonal block as the rows of
//   X = L^{-T} (X L' = I is the same forward substitution as Z' L' = Y'; the tensor-memory row they reuse is the upper
//   triangle of S, which its own panel's update brings to zero).  As rows of the B operand of the rank-8 updates they
//   subtract Z'[n,p] X[r,p]' from column r of the rows of Z' once that column has been consumed, so that after the
//   last panel columns 0..63 of lanes 64..127 hold -Z' L^{-1} = K_t': the gains fall out of the factorisation's own
//   updates, in their error-compensated arithmetic (Z' keeps its low part for this), with no backward solve.
//   (4) then follows the read-out of K_t'.
// Tensor memory of a warpgroup (128 columns): R_W = W, R_F = F (then K_t' on lanes 64..127), then DP.
// Shared memory of a warpgroup: X1 (L in fp32 at the last step when only u_0 is wanted; scratch of the periodic
// symmetrisation) | X0 (P, then Z') | panel hi | panel lo | scratch.  X1 directly precedes X0: step (5) starts its A
// operand 64 rows before Z' so that Z' lands on lanes 64..127 (what the first 64 rows multiply goes to lanes that are
// never read).
//
// Shared-memory operands use the canonical K-major layout without swizzle: 8 x 4 (rows x k) core
// matrices of 128 contiguous bytes, chunk stride 128 B along k, 2048 B between 8-row groups (256 B in the panel
// buffers).  A row owner writes its row with conflict-free 16-byte stores.
//
// Every wait on an MMA-completion barrier is bounded; on a timeout the warpgroup records an error,
// the CTA stops taking work and the kernel still releases tensor memory before it returns.
#pragma once

#include "common.cuh"

namespace ttc {
namespace umma64 {

constexpr int N = 64;
constexpr int WG_THREADS = 128;
constexpr uint32_t SC = 128;                    // bytes between consecutive 4-wide k chunks
constexpr uint32_t SR = 2048;                   // bytes between 8-row groups (16 chunks)
constexpr uint32_t MAT_BYTES = 8 * SR;          // one 64 x 64 matrix
constexpr uint32_t BUF_BYTES = 2 * MAT_BYTES;   // 128 rows
constexpr int SPIN_LIMIT = 1 << 22;

constexpr uint32_t PSR = 256;                   // bytes between 8-row groups of a panel buffer (2 chunks)
constexpr uint32_t PAN_BYTES = 16 * PSR;        // one 128 x 8 buffer

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// byte offset of element (r, c) of a row-major matrix stored as 8 x 4 core matrices
__device__ __forceinline__ uint32_t toff(int r, int c)
{
    return (uint32_t)(r >> 3) * SR + (uint32_t)(c >> 2) * SC + (uint32_t)(r & 7) * 16u + (uint32_t)(c & 3) * 4u;
}
// Private variant of the layout for matrices that are read and updated by the factorisation (S, and the columns
// of Y' that are still being updated): in odd k-chunks the 8 rows of a core matrix are rotated by 4.  The 8-byte
// accumulator-tile accesses of the mma updates (row g, columns 2t, 2t+1: two lanes 128 B apart) then hit
// different banks; row owners (16 bytes) and fragment loads (4 bytes) stay conflict-free.
__device__ __forceinline__ uint32_t toff_rot(int r, int c)
{
    return (uint32_t)(r >> 3) * SR + (uint32_t)(c >> 2) * SC + (uint32_t)(((r & 7) + (((c >> 2) & 1) << 2)) & 7) * 16u +
           (uint32_t)(c & 3) * 4u;
}
__device__ __forceinline__ float& elem(unsigned char* base, uint32_t off) { return *reinterpret_cast<float*>(base + off); }

// fp32 -> tf32 (10 explicit mantissa bits), round to nearest with ties away from zero, on the integer
// pipe (cvt.rna.tf32.f32 issues on the transcendental pipe at a fraction of the rate).
__device__ __forceinline__ uint32_t to_tf32(float x)
{
    return (__float_as_uint(x) + 0x1000u) & 0xffffe000u;
}
__device__ __forceinline__ float round_tf32(float x) { return __uint_as_float(to_tf32(x)); }

// ---- tcgen05 wrappers ---------------------------------------------------------------------------------
// shared-memory matrix descriptor: K-major, no swizzle; `saddr` = address of the first core matrix of
// this k step (a k step of 8 tf32 values spans 2 chunks)
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)(SC >> 4) << 16) | ((uint64_t)(SR >> 4) << 32) |
           ((uint64_t)1 << 46);
}
// the same for a 128 x 8 panel buffer (8-row groups 256 B apart)
__device__ __forceinline__ uint64_t panel_desc(uint32_t saddr)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)(SC >> 4) << 16) | ((uint64_t)(PSR >> 4) << 32) |
           ((uint64_t)1 << 46);
}
// instruction descriptor: tf32 x tf32 -> f32, both operands K-major, M = 128
__device__ __forceinline__ uint32_t instr_desc(int ncols, int negate_a)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)negate_a << 13) | ((uint32_t)(ncols >> 3) << 17) |
           ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}\n"
                 :: "r"(d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}\n"
                 :: "r"(d), "r"(a_tmem), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
// D (128 x ncols) (+)= A (smem, 128 x 64) * B' (smem, ncols x 64), 8 k steps
__device__ __forceinline__ void gemm_ss(uint32_t d, uint32_t a_smem, uint32_t b_smem, int ncols, int negate_a, bool accumulate)
{
    const uint32_t id = instr_desc(ncols, negate_a);
#pragma unroll
    for (int j = 0; j < 8; ++j)
        mma_ss(d, smem_desc(a_smem + 2 * j * SC), smem_desc(b_smem + 2 * j * SC), id, (accumulate || j > 0) ? 1u : 0u);
}
// D (128 x ncols) = A (tensor memory, 128 lanes x 64 columns) * B' (smem, ncols x 64)
__device__ __forceinline__ void gemm_ts(uint32_t d, uint32_t a_tmem, uint32_t b_smem, int ncols)
{
    const uint32_t id = instr_desc(ncols, 0);
#pragma unroll
    for (int j = 0; j < 8; ++j)
        mma_ts(d, a_tmem + 8 * j, smem_desc(b_smem + 2 * j * SC), id, j > 0 ? 1u : 0u);
}
__device__ __forceinline__ void mma_commit(uint32_t mbar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(mbar) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint32_t mbar, uint32_t parity, int limit = SPIN_LIMIT)
{
    for (int it = 0; it < limit; ++it) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                     : "=r"(ok) : "r"(mbar), "r"(parity) : "memory");
        if (ok)
            return true;
    }
    return false;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void async_proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 32 lanes x 32 consecutive columns of tensor memory -> 32 registers per thread (lane = row)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32])
{
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i)
        v[i] = __uint_as_float(r[i]);
}

// 32 lanes x 8 consecutive columns; the caller waits with tmem_wait_ld() before it reads v
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
}
// 32 lanes x 16 consecutive columns; the caller waits with tmem_wait_ld() before it reads r
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 16 registers per thread -> 32 lanes x 16 consecutive columns; followed by tmem_wait_st() before anything depends on it
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                    "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// named barriers: 1 + wg = warps 0, 1 of a warpgroup (64 threads), 5 + wg = the whole warpgroup
__device__ __forceinline__ void half_barrier(int wg) { asm volatile("bar.sync %0, %1;" :: "r"(1 + wg), "r"(64) : "memory"); }
__device__ __forceinline__ void wg_barrier(int wg) { asm volatile("bar.sync %0, %1;" :: "r"(5 + wg), "r"(WG_THREADS) : "memory"); }

// ---- blocked Cholesky of S fused with the forward substitution Z' = Y' L^{-T} --------------------------------------
// In-thread Cholesky of an 8 x 8 SPD block: l (lower triangle) is overwritten by L, rinv[i] = 1 / L[i][i].
// Right-looking; the chain from one pivot to the next is rsqrt -> multiply -> fma.
// Returns 0 or 1 + the index of the first non-positive pivot.
__device__ __forceinline__ int chol8(float (&l)[8][8], float (&rinv)[8])
{
    int bad = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float d = l[j][j];
        if (!(d > 0.f)) {
            if (!bad)
                bad = j + 1;
            d = 1.f;
        }
        float rs;
        asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(rs) : "f"(d));
        rinv[j] = rs;
#pragma unroll
        for (int i = j + 1; i < 8; ++i)
            l[i][j] *= rs;
#pragma unroll
        for (int i = j + 1; i < 8; ++i)
#pragma unroll
            for (int c = j + 1; c <= i; ++c)
                l[i][c] = fmaf(-l[i][j], l[c][j], l[i][c]);
        l[j][j] = d * rs;
    }
    return bad;
}
// x (a row vector of 8) <- x L^{-T}  (forward substitution with the lower factor L)
__device__ __forceinline__ void fsub8(float (&x)[8], const float (&l)[8][8], const float (&rinv)[8])
{
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float v = x[i];
#pragma unroll
        for (int j = 0; j < i; ++j)
            v = fmaf(-l[i][j], x[j], v);
        x[i] = v * rinv[i];
    }
}
// 8 consecutive columns (an even chunk and the odd chunk after it) of one row.  `grp` points at the even chunk
// of the row's 8-row group, `slot` = row & 7.  ROT: rotated layout (odd chunk at slot + 4), else canonical.
template <bool ROT>
__device__ __forceinline__ void load_row8(float (&x)[8], const unsigned char* grp, int slot)
{
    const float4 a = *reinterpret_cast<const float4*>(grp + slot * 16);
    const float4 b = *reinterpret_cast<const float4*>(grp + SC + (ROT ? ((slot + 4) & 7) : slot) * 16);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
template <bool ROT, bool ROUND>
__device__ __forceinline__ void store_row8(unsigned char* grp, int slot, const float (&x)[8])
{
    float4 a = make_float4(x[0], x[1], x[2], x[3]), b = make_float4(x[4], x[5], x[6], x[7]);
    if (ROUND) {
        a.x = round_tf32(a.x); a.y = round_tf32(a.y); a.z = round_tf32(a.z); a.w = round_tf32(a.w);
        b.x = round_tf32(b.x); b.y = round_tf32(b.y); b.z = round_tf32(b.z); b.w = round_tf32(b.w);
    }
    *reinterpret_cast<float4*>(grp + slot * 16) = a;
    *reinterpret_cast<float4*>(grp + SC + (ROT ? ((slot + 4) & 7) : slot) * 16) = b;
}

// ---- global-memory helpers --------------------------------------------------------------------------------------
__device__ __forceinline__ void wg_fail_instance(const SolveParams& p, long long inst, int code, int wt)
{
    const float qn = quiet_nan();
    const int H = p.H;
    const int obf = p.out_bf16;
    if (p.K)
        for (long long e = wt; e < (long long)H * N * N; e += WG_THREADS)
            store_out(p.K, inst * (long long)H * N * N + e, qn, obf);
    if (p.P) {
        const long long cnt = (long long)(p.first_only ? 1 : H + 1) * N * N;
        for (long long e = wt; e < cnt; e += WG_THREADS)
            store_out(p.P, inst * cnt + e, qn, obf);
    }
    if (p.x)
        for (long long e = wt; e < (long long)(H + 1) * N; e += WG_THREADS)
            store_out(p.x, inst * (long long)(H + 1) * N + e, qn, obf);
    if (p.u) {
        const long long cnt = p.first_only ? N : (long long)H * N;
        for (long long e = wt; e < cnt; e += WG_THREADS)
            store_out(p.u, inst * cnt + e, qn, obf);
    }
    if (p.info && wt == 0)
        p.info[inst] = code;
}

constexpr int NUM_WG = 4;
constexpr int THREADS = NUM_WG * WG_THREADS;
constexpr int TOK = 8;                                  // tokens per warpgroup and work item
constexpr int CHUNK = NUM_WG * TOK;                   // tokens per work item of a CTA
constexpr uint32_t OFF_X1 = 0;
constexpr uint32_t OFF_X0 = MAT_BYTES;
constexpr uint32_t OFF_PH = 2 * MAT_BYTES;
constexpr uint32_t OFF_PL = 2 * MAT_BYTES + PAN_BYTES;
constexpr uint32_t OFF_MISC = 2 * MAT_BYTES + 2 * PAN_BYTES;
struct Misc {
    unsigned long long mbar;     // MMA completion barrier (every thread waits on it)
    unsigned long long mbar_w;   // completion of W = BA P': only the issuing thread waits on it
    int dead;                    // set when a wait timed out
    int flag;                    // first failed pivot (0 = none)
    alignas(16) float x0[N];
    alignas(16) float y0[N];     // Y x_0 / u_t of the rollout; during the factorisation: the 8 x 8 diagonal block
    alignas(16) float ld[36];    // current diagonal factor: strict lower triangle (28) + reciprocal pivots (8)
};
constexpr uint32_t WG_BYTES = OFF_MISC + ((sizeof(Misc) + 127) / 128) * 128;
struct CtaShared {
    int chunk;                   // current work item
    int dead;                    // some warpgroup gave up: the CTA stops taking work
    uint32_t tmem_base;
};
constexpr int R_LD = N + 4;                                // row stride of R in shared memory (conflict-free row owners)
constexpr uint32_t R_BYTES = N * R_LD * 4;
constexpr uint32_t SMEM_BYTES = BUF_BYTES + R_BYTES + NUM_WG * WG_BYTES + 128;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");


// half a row (32 values) of the Q matrix of one instance
__device__ __forceinline__ void load_q_half(float (&q)[32], const OperandDev& Q, long long oq, int j, int half)
{
    if (Q.dtype == TTC_BF16) {
        const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(Q.ptr) + oq + (long long)j * N + 32 * half);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint4 v = __ldg(src + c);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                q[8 * c + 2 * e] = __uint_as_float(w[e] << 16);
                q[8 * c + 2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
            }
        }
    } else {
        const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(Q.ptr) + oq + (long long)j * N + 32 * half);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const float4 v = __ldg(src + c);
            q[4 * c] = v.x; q[4 * c + 1] = v.y; q[4 * c + 2] = v.z; q[4 * c + 3] = v.w;
        }
    }
}
// columns 32 half .. 32 half + 31 of row `r` of a 64-row operand <- values rounded to tf32
__device__ __forceinline__ void store_half_tf32(unsigned char* buf, int r, int half, const float (&v)[32])
{
#pragma unroll
    for (int c = 0; c < 8; ++c)
        *reinterpret_cast<float4*>(buf + toff(r, 32 * half + 4 * c)) =
            make_float4(round_tf32(v[4 * c]), round_tf32(v[4 * c + 1]), round_tf32(v[4 * c + 2]), round_tf32(v[4 * c + 3]));
}
// 32 consecutive output elements starting at element `idx` of `base` (float32 or bfloat16 output)
__device__ __forceinline__ void store_half_global(float* base, long long idx, const float (&v)[32], int bf16)
{
#pragma unroll
    for (int c = 0; c < 8; ++c)
        store_out4(base, idx + 4 * c, make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]), bf16);
}

// GAINS = the request needs every K_t (K, x or the full u wanted); the other instantiation carries none of that code.
template <bool GAINS>
__global__ void __launch_bounds__(THREADS, 1) riccati_umma64_kernel(SolveParams p, int* chunk_counter, int* error_flag)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const int tid = threadIdx.x;
    const int wg = tid / WG_THREADS;
    const int wt = tid % WG_THREADS;
    const int warp = wt >> 5;                  // warp in warpgroup: owns tensor-memory lanes 32 warp .. 32 warp + 31
    const int lane = wt & 31;
    unsigned char* BA = smem_raw;              // rows 0..63: B' (row j = column j of B), rows 64..127: A'; shared by the CTA
    float* Rs = reinterpret_cast<float*>(smem_raw + BUF_BYTES);   // R of the head, fp32, shared by the CTA
    unsigned char* wsm = smem_raw + BUF_BYTES + R_BYTES + (size_t)wg * WG_BYTES;
    unsigned char* X1 = wsm + OFF_X1;        // L in fp32 for u_0 at the last step; scratch of the mirror and of the symmetrisation
    unsigned char* X0 = wsm + OFF_X0;        // P -> Z' -> next P
    unsigned char* PH = wsm + OFF_PH;        // panel operand, hi parts (128 x 8)
    unsigned char* PL = wsm + OFF_PL;        // panel operand, lo parts
    Misc& misc = *reinterpret_cast<Misc*>(wsm + OFF_MISC);
    CtaShared& cta = *reinterpret_cast<CtaShared*>(smem_raw + BUF_BYTES + R_BYTES + (size_t)NUM_WG * WG_BYTES);
    const uint32_t mbar = smem_u32(&misc.mbar);
    const uint32_t mbar_w = smem_u32(&misc.mbar_w);

    if (wt == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(mbar) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(mbar_w) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        misc.dead = 0;
    }
    if (tid == 0)
        cta.dead = 0;
    // rows 64..127 (Z') of the low-part panel buffer stay zero: Z' is kept as tf32
    if (wt >= 64)
        for (int e = wt - 64; e < 128; e += 64)
            *reinterpret_cast<float4*>(PL + 8u * PSR + (uint32_t)e * 16u) = make_float4(0.f, 0.f, 0.f, 0.f);
    async_proxy_fence();
    if (tid < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&cta.tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t RW = cta.tmem_base + 128u * wg, RF = RW + 64u;
    const uint32_t lane_sel = (uint32_t)(32 * warp) << 16;
    uint32_t parity = 0, parity_w = 0;
    const bool issuer = wt == 96;              // one thread of warp 3 issues every MMA of the warpgroup

    const int H = p.H;
    const long long chunks_per_head = (p.tcount + CHUNK - 1) / CHUNK;
    const long long nchunks = p.b0 * p.b1 * chunks_per_head;
    constexpr bool need_K_all = GAINS;
    const bool want_u0 = (p.u != nullptr) && p.first_only && !need_K_all;
    // With bfloat16 outputs the rollout kernel still reads float32 gains: they go to the workspace, and to K as
    // bfloat16 too.
    const int obf = p.out_bf16;
    float* Kbase = (p.K && !obf) ? p.K : p.Kws;
    long long offA_loaded = -1, offB_loaded = -1, offR_loaded = -1;
    bool dead = false;

    auto wait_mma = [&]() {
        if (!mbar_wait(mbar, parity)) {
            misc.dead = 1;
            atomicExch(error_flag, 1);
        }
        parity ^= 1u;
        tc_fence_after();
    };

    for (;;) {
        if (dead)
            cta.dead = 1;
        __syncthreads();                       // every warpgroup is done with BA and with the last work item
        if (tid == 0)
            cta.chunk = atomicAdd(chunk_counter, 1);
        __syncthreads();
        const long long chunk = cta.chunk;
        if (chunk >= nchunks || cta.dead)
            break;
        const long long head = chunk / chunks_per_head;
        const long long tok0 = p.t0 + (chunk % chunks_per_head) * CHUNK;
        const long long inst0 = head * p.b2 + tok0;
        const int ntok = (int)min((long long)CHUNK, p.t0 + p.tcount - tok0);
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
                    elem(BA, toff(j, k)) = round_tf32(__ldg(Bg + e));
                    elem(BA, toff(64 + j, k)) = round_tf32(__ldg(Ag + e));
                    Rs[k * R_LD + j] = __ldg(Rg + e);
                }
                offA_loaded = oa; offB_loaded = ob; offR_loaded = orr;
                async_proxy_fence();
                __syncthreads();
            }
        }
        const int my0 = TOK * wg, my1 = min(ntok, TOK * wg + TOK);

        for (int tk = my0; tk < my1 && !dead; ++tk) {
            const long long inst = inst0 + tk;
            const long long oq = operand_offset(p.Q, inst, p.b1, p.b2);
            // ---- P_H = Q: warps 2, 3 own the rows of the value matrix
            if (warp >= 2) {
                const int j = wt - 64;
#pragma unroll 1
                for (int half = 0; half < 2; ++half) {
                    float q[32];
                    load_q_half(q, p.Q, oq, j, half);
                    store_half_tf32(X0, j, half, q);
                    if (p.P && !p.first_only)
                        store_half_global(p.P, (inst * (long long)(H + 1) + H) * N * N + (long long)j * N + 32 * half, q, obf);
                }
            } else if (p.x0.ptr && warp == 0) {
                const long long ox = operand_offset(p.x0, inst, p.b1, p.b2);
                misc.x0[2 * lane] = load_elem(p.x0, ox + 2 * lane);
                misc.x0[2 * lane + 1] = load_elem(p.x0, ox + 2 * lane + 1);
            }
            if (wt == 0)
                misc.flag = 0;
            async_proxy_fence();
            wg_barrier(wg);

            for (int ts = H - 1; ts >= 0 && !dead; --ts) {
                // (1) W = BA P' -> R_W ; (2) F = W B -> R_F
                if (issuer) {
                    tc_fence_after();
                    gemm_ss(RW, smem_u32(BA), smem_u32(X0), 64, 0, false);
                    // F reads W from tensor memory: an MMA whose A operand was written by the MMAs just before it is NOT
                    // ordered after them by the pipe (measured: 7 % error in F when chained), so the issuing thread
                    // waits for W on a barrier of its own before it issues F
                    mma_commit(mbar_w);
                    if (!mbar_wait(mbar_w, parity_w)) {
                        misc.dead = 1;
                        atomicExch(error_flag, 1);
                    }
                    parity_w ^= 1u;
                    tc_fence_after();
                    gemm_ts(RF, RW, smem_u32(BA), 64);
                    mma_commit(mbar);
                }
                wait_mma();
                // (3) [S; Y'] = [L; Z'] L' panel by panel, thread wt owns row wt
                const bool keep_l = ts == 0 && want_u0;        // fp32 copy of L for the back substitution of u_0
                float* diag = &misc.y0[0];                     // [8][8]
                float v[8];
                auto load_cols = [&](int c0) {
                    uint32_t raw[8];
                    tmem_ld8(RF + lane_sel + c0, raw);
                    float4 r0 = make_float4(0.f, 0.f, 0.f, 0.f), r1 = r0;
                    if (warp < 2) {
                        r0 = *reinterpret_cast<const float4*>(Rs + wt * R_LD + c0);
                        r1 = *reinterpret_cast<const float4*>(Rs + wt * R_LD + c0 + 4);
                    }
                    tmem_wait_ld();
                    v[0] = __uint_as_float(raw[0]) + r0.x; v[1] = __uint_as_float(raw[1]) + r0.y;
                    v[2] = __uint_as_float(raw[2]) + r0.z; v[3] = __uint_as_float(raw[3]) + r0.w;
                    v[4] = __uint_as_float(raw[4]) + r1.x; v[5] = __uint_as_float(raw[5]) + r1.y;
                    v[6] = __uint_as_float(raw[6]) + r1.z; v[7] = __uint_as_float(raw[7]) + r1.w;
                };
                if (GAINS && warp < 2) {
                    // The rows of L^{-T} start from the upper triangle of S, the factorisation reads the lower one, and
                    // the two differ by the rounding of the tf32 contractions (and of a P that is only symmetrised now
                    // and then): at 1e-3 of |S| that would be the error of the gains.  Mirror the lower triangle into
                    // the upper one first: every row through X1 (free here), element (r, c) at word 64 r + (c ^ r) so
                    // that both the row stores and the column reads touch 32 banks.
                    float* tr = reinterpret_cast<float*>(X1);
#pragma unroll
                    for (int qt = 0; qt < 4; ++qt) {
                        uint32_t raw[16];
                        tmem_ld16(RF + lane_sel + 16 * qt, raw);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 16; ++c)
                            tr[64 * wt + ((16 * qt + c) ^ wt)] = __uint_as_float(raw[c]);
                    }
                    half_barrier(wg);
#pragma unroll
                    for (int qt = 0; qt < 4; ++qt) {
                        uint32_t raw[16];
                        tmem_ld16(RF + lane_sel + 16 * qt, raw);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const int cc = 16 * qt + c;
                            if (cc > wt)
                                raw[c] = __float_as_uint(tr[64 * cc + (wt ^ cc)]);
                        }
                        tmem_st16(RF + lane_sel + 16 * qt, raw);
                    }
                    tmem_wait_st();
                }
                load_cols(0);
#pragma unroll 1
                for (int pnl = 0; pnl < 8; ++pnl) {
                    const int col = 8 * pnl;
                    if (warp == (pnl >> 2)) {
                        // the 8 rows of the diagonal block belong to this warp: gather the block, factor it (every
                        // lane redundantly) and publish L_d and the reciprocal pivots
                        if ((unsigned)(wt - col) < 8u) {
                            float4* dst = reinterpret_cast<float4*>(diag + 8 * (wt - col));
                            dst[0] = make_float4(v[0], v[1], v[2], v[3]);
                            dst[1] = make_float4(v[4], v[5], v[6], v[7]);
                        }
                        __syncwarp();
                        float l[8][8], rinv[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float4 a4 = *reinterpret_cast<const float4*>(diag + 8 * i);
                            const float4 b4 = *reinterpret_cast<const float4*>(diag + 8 * i + 4);
                            l[i][0] = a4.x; l[i][1] = a4.y; l[i][2] = a4.z; l[i][3] = a4.w;
                            l[i][4] = b4.x; l[i][5] = b4.y; l[i][6] = b4.z; l[i][7] = b4.w;
                        }
                        const int bad = chol8(l, rinv);
                        if (lane == 0) {
                            float4* dst = reinterpret_cast<float4*>(&misc.ld[0]);
                            dst[0] = make_float4(l[1][0], l[2][0], l[2][1], l[3][0]);
                            dst[1] = make_float4(l[3][1], l[3][2], l[4][0], l[4][1]);
                            dst[2] = make_float4(l[4][2], l[4][3], l[5][0], l[5][1]);
                            dst[3] = make_float4(l[5][2], l[5][3], l[5][4], l[6][0]);
                            dst[4] = make_float4(l[6][1], l[6][2], l[6][3], l[6][4]);
                            dst[5] = make_float4(l[6][5], l[7][0], l[7][1], l[7][2]);
                            dst[6] = make_float4(l[7][3], l[7][4], l[7][5], l[7][6]);
                            dst[7] = make_float4(rinv[0], rinv[1], rinv[2], rinv[3]);
                            dst[8] = make_float4(rinv[4], rinv[5], rinv[6], rinv[7]);
                            if (bad && misc.flag == 0)
                                misc.flag = ts * N + col + bad;
                        }
                    }
                    tc_fence_before();
                    wg_barrier(wg);
                    if (misc.dead != 0) {
                        dead = true;
                        break;
                    }
                    if (!GAINS && pnl == 7 && issuer) {
                        // every row has read its last columns of F: (4) DP = W A into the columns of F
                        // (with gains the columns of F still collect K_t': (4) follows their read-out)
                        tc_fence_after();
                        gemm_ts(RF, RW, smem_u32(BA) + MAT_BYTES, 64);
                    }
                    // GAINS: rows 0..63 carry X = L^{-T} behind L.  Row r of L ends in its diagonal block; from there on the
                    // same tensor-memory row (the unused upper triangle of S, which the trailing updates have brought to
                    // L[r,p] L[c,p]' = what this panel's update removes) is continued as row r of X (X L' = I is the
                    // substitution the rows of Z' go through): in the diagonal panel the operand row is
                    // L[r,p] + e_r L_d^{-T}, afterwards it is the row read back from tensor memory, substituted.
                    // These rows are also rows of the B operand, so the trailing updates keep subtracting
                    // Z'[n,p] X[r,p]' from column r of the rows of Z' after that column has been consumed (and brought to
                    // zero by its own panel): when the last panel is done, columns 0..63 of lanes 64..127 hold
                    // -Z' X' = -Z' L^{-1} = K_t', in the error-compensated arithmetic of the updates.  No backward solve.
                    float xi[8];                               // diagonal panel: row wt - col of L_d^{-T} (GAINS, warps 0, 1)
                    {
                        float l[8][8], rinv[8];
                        const float4* src = reinterpret_cast<const float4*>(&misc.ld[0]);
                        const float4 c0 = src[0], c1 = src[1], c2 = src[2], c3 = src[3], c4 = src[4], c5 = src[5],
                                     c6 = src[6], c7 = src[7], c8 = src[8];
                        l[1][0] = c0.x; l[2][0] = c0.y; l[2][1] = c0.z; l[3][0] = c0.w;
                        l[3][1] = c1.x; l[3][2] = c1.y; l[4][0] = c1.z; l[4][1] = c1.w;
                        l[4][2] = c2.x; l[4][3] = c2.y; l[5][0] = c2.z; l[5][1] = c2.w;
                        l[5][2] = c3.x; l[5][3] = c3.y; l[5][4] = c3.z; l[6][0] = c3.w;
                        l[6][1] = c4.x; l[6][2] = c4.y; l[6][3] = c4.z; l[6][4] = c4.w;
                        l[6][5] = c5.x; l[7][0] = c5.y; l[7][1] = c5.z; l[7][2] = c5.w;
                        l[7][3] = c6.x; l[7][4] = c6.y; l[7][5] = c6.z; l[7][6] = c6.w;
                        rinv[0] = c7.x; rinv[1] = c7.y; rinv[2] = c7.z; rinv[3] = c7.w;
                        rinv[4] = c8.x; rinv[5] = c8.y; rinv[6] = c8.z; rinv[7] = c8.w;
                        fsub8(v, l, rinv);
                        if (GAINS && warp < 2) {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                xi[j] = 0.f;
                            if (warp == (pnl >> 2)) {          // the warp of the diagonal block: row (wt - col) of L_d^{-T}
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    xi[j] = (col + j == wt) ? 1.f : 0.f;
                                fsub8(xi, l, rinv);
                            }
                        }
                    }
                    {
                        unsigned char* ph = PH + (uint32_t)(wt >> 3) * PSR + (uint32_t)(wt & 7) * 16u;
                        float hi[8];
                        if (warp < 2) {                        // row wt of L: lower triangular, ends at column wt
                            float lo[8];
                            if (GAINS) {
                                const bool done = wt < col;    // finished row: v is its row of L^{-T}
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    if (!done && col + j > wt)
                                        v[j] = 0.f;
#pragma unroll
                                for (int j = 0; j < 8; ++j) {
                                    const float a = done ? v[j] : v[j] + xi[j];
                                    hi[j] = round_tf32(a);
                                    lo[j] = a - hi[j];
                                }
                            } else {
#pragma unroll
                                for (int j = 0; j < 8; ++j) {
                                    if (col + j > wt)
                                        v[j] = 0.f;
                                    hi[j] = round_tf32(v[j]);
                                    lo[j] = v[j] - hi[j];
                                }
                            }
                            unsigned char* pl = PL + (uint32_t)(wt >> 3) * PSR + (uint32_t)(wt & 7) * 16u;
                            *reinterpret_cast<float4*>(pl) = make_float4(lo[0], lo[1], lo[2], lo[3]);
                            *reinterpret_cast<float4*>(pl + SC) = make_float4(lo[4], lo[5], lo[6], lo[7]);
                            if (keep_l)                        // fp32 copy for u_0
                                store_row8<true, false>(X1 + (uint32_t)(wt >> 3) * SR + 2u * pnl * SC, wt & 7, v);
                        } else {                               // row wt - 64 of Z': tf32 as operand of (5)
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                hi[j] = round_tf32(v[j]);
                            if (GAINS) {                       // the gains collect in the updates: keep the low part too
                                unsigned char* pl = PL + (uint32_t)(wt >> 3) * PSR + (uint32_t)(wt & 7) * 16u;
                                *reinterpret_cast<float4*>(pl) = make_float4(v[0] - hi[0], v[1] - hi[1], v[2] - hi[2], v[3] - hi[3]);
                                *reinterpret_cast<float4*>(pl + SC) = make_float4(v[4] - hi[4], v[5] - hi[5], v[6] - hi[6], v[7] - hi[7]);
                            }
                            unsigned char* pz = X0 + (uint32_t)((wt - 64) >> 3) * SR + 2u * pnl * SC + (uint32_t)(wt & 7) * 16u;
                            *reinterpret_cast<float4*>(pz) = make_float4(hi[0], hi[1], hi[2], hi[3]);
                            *reinterpret_cast<float4*>(pz + SC) = make_float4(hi[4], hi[5], hi[6], hi[7]);
                        }
                        *reinterpret_cast<float4*>(ph) = make_float4(hi[0], hi[1], hi[2], hi[3]);
                        *reinterpret_cast<float4*>(ph + SC) = make_float4(hi[4], hi[5], hi[6], hi[7]);
                    }
                    if (pnl == 7 && !GAINS)
                        break;
                    async_proxy_fence();
                    wg_barrier(wg);
                    if (issuer) {                              // G -= panel * panel[0:64]'  (hi*hi + lo*hi + hi*lo)
                        tc_fence_after();
                        const uint32_t idn = instr_desc(64, 1);
                        const uint64_t dh = panel_desc(smem_u32(PH)), dl = panel_desc(smem_u32(PL));
                        mma_ss(RF, dh, dh, idn, 1u);
                        mma_ss(RF, dl, dh, idn, 1u);
                        mma_ss(RF, dh, dl, idn, 1u);
                        mma_commit(mbar);
                    }
                    wait_mma();
                    if (pnl == 7)
                        break;
                    load_cols(col + 8);
                }
                if (GAINS && warp >= 2 && !dead && misc.dead == 0) {
                    // K_t' from the columns of F (lanes 64..127): thread 64 + n holds K_t[:, n]
                    const int nn = wt - 64;
                    const long long ko = (inst * (long long)H + ts) * N * N + nn;
#pragma unroll
                    for (int qt = 0; qt < 4; ++qt) {
                        uint32_t raw[16];
                        tmem_ld16(RF + lane_sel + 16 * qt, raw);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const float kv = __uint_as_float(raw[c]);
                            Kbase[ko + (long long)(16 * qt + c) * N] = kv;
                            if (obf && p.K)
                                store_out(p.K, ko + (long long)(16 * qt + c) * N, kv, 1);
                        }
                    }
                }
                async_proxy_fence();
                tc_fence_before();
                wg_barrier(wg);
                dead = dead || misc.dead != 0;
                // (5) DP -= Z' Z : A operand rows 64..127 = Z' (rows 0..63 = X1, unused lanes)
                if (issuer && !dead) {
                    tc_fence_after();
                    if (GAINS)                                 // (4), once K_t' has been read out of the columns of F
                        gemm_ts(RF, RW, smem_u32(BA) + MAT_BYTES, 64);
                    gemm_ss(RF, smem_u32(X0) - MAT_BYTES, smem_u32(X0), 64, 1, true);
                    mma_commit(mbar);
                }
                if (dead)
                    break;
                // Without gains nothing else runs between here and the read-out: the row of Q that the read-out adds
                // travels while (5) is in flight (bf16: the whole row in 32 registers).
                uint4 qraw[8];
                const bool q_pref = !GAINS && p.Q.dtype == TTC_BF16;
                if (q_pref && warp >= 2) {
                    const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.Q.ptr) + oq + (long long)(wt - 64) * N);
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        qraw[c] = __ldg(src + c);
                }
                if (ts == 0 && want_u0 && warp < 2) {
                    // u_0 = K_0 x_0 = -L^{-T} (Z x_0), fp32, by the 64 threads of warps 0, 1
                    const int i = wt;
                    half_barrier(wg);
                    float zi = 0.f;
#pragma unroll 8
                    for (int c = 0; c < N; ++c)
                        zi = fmaf(elem(X0, toff(c, i)), misc.x0[c], zi);               // Z[i][c] = Z'[c][i]
                    misc.y0[i] = zi;
#pragma unroll 1
                    for (int kb = 7; kb >= 0; --kb) {           // back substitution L' w = Z x_0 in 8-wide blocks
                        half_barrier(wg);
                        const int c0 = 8 * kb;
                        float l[8][8], w[8];
#pragma unroll
                        for (int r = 0; r < 8; ++r) {
                            load_row8<true>(l[r], X1 + toff(c0, c0), r);
                            w[r] = misc.y0[c0 + r];
                        }
#pragma unroll
                        for (int r = 7; r >= 0; --r) {
                            float vv = w[r];
#pragma unroll
                            for (int j = r + 1; j < 8; ++j)
                                vv = fmaf(-l[j][r], w[j], vv);
                            w[r] = vv / l[r][r];
                        }
                        if (i < c0) {
#pragma unroll
                            for (int r = 0; r < 8; ++r)
                                zi = fmaf(-elem(X1, toff_rot(c0 + r, i)), w[r], zi);
                        }
                        half_barrier(wg);
                        if (i < c0)
                            misc.y0[i] = zi;
#pragma unroll
                        for (int r = 0; r < 8; ++r)
                            if (i == c0 + r)
                                store_out(p.u, inst * (long long)N + i, -w[r], obf);
                    }
                }
                wait_mma();
                // P_t = Q + DP: warps 2, 3 own the rows (lanes 64..127)
                if (warp >= 2) {
                    const int j = wt - 64;
                    const bool Pdst = p.P && (!p.first_only || ts == 0);
                    const long long Pidx = (inst * (long long)(p.first_only ? 1 : H + 1) + (p.first_only ? 0 : ts)) * N * N + (long long)j * N;
                    if (q_pref) {
#pragma unroll
                        for (int qt = 0; qt < 4; ++qt) {       // 16 columns at a time
                            float q[16];
#pragma unroll
                            for (int c = 0; c < 2; ++c) {
                                const uint4 v4 = qraw[2 * qt + c];
                                const uint32_t wd[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    q[8 * c + 2 * e] = __uint_as_float(wd[e] << 16);
                                    q[8 * c + 2 * e + 1] = __uint_as_float(wd[e] & 0xffff0000u);
                                }
                            }
                            uint32_t raw[16];
                            tmem_ld16(RF + lane_sel + 16 * qt, raw);
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 16; ++c)
                                q[c] += __uint_as_float(raw[c]);
                            if (ts > 0) {
#pragma unroll
                                for (int c = 0; c < 4; ++c)
                                    *reinterpret_cast<float4*>(X0 + toff(j, 16 * qt + 4 * c)) =
                                        make_float4(round_tf32(q[4 * c]), round_tf32(q[4 * c + 1]), round_tf32(q[4 * c + 2]), round_tf32(q[4 * c + 3]));
                            }
                            if (Pdst) {
#pragma unroll
                                for (int c = 0; c < 4; ++c)
                                    store_out4(p.P, Pidx + 16 * qt + 4 * c, make_float4(q[4 * c], q[4 * c + 1], q[4 * c + 2], q[4 * c + 3]), obf);
                            }
                        }
                    } else {
#pragma unroll 1
                        for (int half = 0; half < 2; ++half) {
                            float q[32], hh[32];
                            load_q_half(q, p.Q, oq, j, half);
                            tmem_ld32(RF + lane_sel + 32 * half, hh);
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                q[c] += hh[c];
                            if (ts > 0)
                                store_half_tf32(X0, j, half, q);
                            if (Pdst)
                                store_half_global(p.P, Pidx + 32 * half, q, obf);
                        }
                    }
                    // Every eighth step the operand is replaced by (P + P') / 2.  Q and Z'Z are symmetric but the rounding
                    // of A'(P A) is not, and the antisymmetric part E obeys E <- A'E A: along an open-loop unstable A it
                    // grows however well the closed loop is damped, until S stops being positive definite.  Eight steps
                    // of growth are harmless (the exchange costs about a sixth of a step).  X1 is free here and takes the averaged rows.
                    if (ts > 0 && (ts & 7) == 0) {
                        half_barrier(wg);                     // both halves of every row are in X0
#pragma unroll 8
                        for (int c = 0; c < 64; ++c) {
                            const int cj = (c + (j >> 2)) & 63;       // rotated per lane: the column reads hit 32 banks
                            elem(X1, toff(j, cj)) = round_tf32(0.5f * (elem(X0, toff(j, cj)) + elem(X0, toff(cj, j))));
                        }
                        half_barrier(wg);                     // every column has been read
#pragma unroll
                        for (int c = 0; c < 16; ++c)
                            *reinterpret_cast<float4*>(X0 + toff(j, 4 * c)) = *reinterpret_cast<const float4*>(X1 + toff(j, 4 * c));
                    }
                }
                tc_fence_before();
                async_proxy_fence();
                wg_barrier(wg);
                dead = dead || misc.dead != 0;
            }
            if (dead)
                break;
            wg_barrier(wg);
            // ---- status / failed instance
            {
                const int fl = misc.flag;
                if (fl) {
                    wg_fail_instance(p, inst, fl, wt);
                    if (need_K_all && wt == 0)               // the rollout kernel skips instances whose first gain is NaN
                        Kbase[inst * (long long)H * N * N] = quiet_nan();
                }
                else if (p.info && wt == 0)
                    p.info[inst] = 0;
            }
            wg_barrier(wg);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (tid < 32)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(cta.tmem_base), "r"(512) : "memory");
}

// ---- forward loop of Alg. 1 for n = m = 64: u_t = K_t x_t, x_{t+1} = A x_t + B u_t (fp32) ---------------------------
// Separate kernel, launched after the backward pass: one warp per instance, 8 warps per CTA on consecutive tokens of
// one head (A, B of the head in shared memory).  K_t (16 KB per step and instance) is streamed from memory exactly
// once with fully coalesced 16-byte loads: lanes 0..15 and 16..31 each take one row per load and the 16 partial dot
// products are reduced with shuffles.  Instances whose first gain is NaN (failed in the backward pass, outputs
// already filled with NaN) are skipped.
constexpr int ROLL_WARPS = 8;
constexpr int ROLL_LD = N + 4;
struct RollSmem {
    float A[N * ROLL_LD], B[N * ROLL_LD];
    float x[ROLL_WARPS][N], u[ROLL_WARPS][N];
};
__global__ void __launch_bounds__(32 * ROLL_WARPS, 5) rollout64_kernel(SolveParams p, const float* Kall)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    RollSmem& sm = *reinterpret_cast<RollSmem*>(smem_raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int H = p.H;
    const long long chunks_per_head = (p.tcount + ROLL_WARPS - 1) / ROLL_WARPS;
    const long long nchunks = p.b0 * p.b1 * chunks_per_head;
    long long offA = -1, offB = -1;
    for (long long chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
        const long long head = chunk / chunks_per_head;
        const long long tok0 = p.t0 + (chunk % chunks_per_head) * ROLL_WARPS;
        const long long inst0 = head * p.b2 + tok0;
        const int ntok = (int)min((long long)ROLL_WARPS, p.t0 + p.tcount - tok0);
        const long long oa = operand_offset(p.A, inst0, p.b1, p.b2), ob = operand_offset(p.B, inst0, p.b1, p.b2);
        __syncthreads();
        if (oa != offA || ob != offB) {
            const float* Ag = reinterpret_cast<const float*>(p.A.ptr) + oa;
            const float* Bg = reinterpret_cast<const float*>(p.B.ptr) + ob;
            for (int e = threadIdx.x; e < N * N; e += 32 * ROLL_WARPS) {
                sm.A[(e >> 6) * ROLL_LD + (e & 63)] = __ldg(Ag + e);
                sm.B[(e >> 6) * ROLL_LD + (e & 63)] = __ldg(Bg + e);
            }
            offA = oa; offB = ob;
        }
        __syncthreads();
        if (warp >= ntok)
            continue;
        const long long inst = inst0 + warp;
        const float* Ki = Kall + inst * (long long)H * N * N;
        if (isnan(__ldg(Ki)))
            continue;
        float* xs = sm.x[warp];
        float* us = sm.u[warp];
        const int obf = p.out_bf16;
        const bool xo = p.x != nullptr, uo = p.u != nullptr;
        const long long xoff = inst * (long long)(H + 1) * N, uoff = inst * (long long)(p.first_only ? 1 : H) * N;
        {
            const long long ox = operand_offset(p.x0, inst, p.b1, p.b2);
            const float a = load_elem(p.x0, ox + lane), b = load_elem(p.x0, ox + lane + 32);
            xs[lane] = a; xs[lane + 32] = b;
            if (xo) { store_out(p.x, xoff + lane, a, obf); store_out(p.x, xoff + lane + 32, b, obf); }
        }
        __syncwarp();
        const int half = lane >> 4, seg = lane & 15;
#pragma unroll 1
        for (int ts = 0; ts < H; ++ts) {
            const float4 x4 = *reinterpret_cast<const float4*>(xs + 4 * seg);
            const float4* Kt = reinterpret_cast<const float4*>(Ki + (long long)ts * N * N) + lane;     // row (lane >> 4), segment (lane & 15)
#pragma unroll 8
            for (int it = 0; it < 32; ++it) {                 // rows 2 it, 2 it + 1
                const float4 k4 = __ldcs(Kt + 32 * it);
                float s = fmaf(k4.x, x4.x, fmaf(k4.y, x4.y, fmaf(k4.z, x4.z, k4.w * x4.w)));
                s += __shfl_xor_sync(0xffffffffu, s, 8);
                s += __shfl_xor_sync(0xffffffffu, s, 4);
                s += __shfl_xor_sync(0xffffffffu, s, 2);
                s += __shfl_xor_sync(0xffffffffu, s, 1);
                if (seg == 0)
                    us[2 * it + half] = s;
            }
            __syncwarp();
            if (uo && (!p.first_only || ts == 0)) {
                const long long ut = uoff + (p.first_only ? 0 : (long long)ts * N);
                store_out(p.u, ut + lane, us[lane], obf);
                store_out(p.u, ut + lane + 32, us[lane + 32], obf);
            }
            float n0 = 0.f, n1 = 0.f;                         // rows lane and lane + 32 of A x + B u
#pragma unroll
            for (int c4 = 0; c4 < 16; ++c4) {
                const float4 xv = *reinterpret_cast<const float4*>(xs + 4 * c4);
                const float4 uv = *reinterpret_cast<const float4*>(us + 4 * c4);
                const float4 a0 = *reinterpret_cast<const float4*>(sm.A + lane * ROLL_LD + 4 * c4);
                const float4 a1 = *reinterpret_cast<const float4*>(sm.A + (lane + 32) * ROLL_LD + 4 * c4);
                const float4 b0 = *reinterpret_cast<const float4*>(sm.B + lane * ROLL_LD + 4 * c4);
                const float4 b1 = *reinterpret_cast<const float4*>(sm.B + (lane + 32) * ROLL_LD + 4 * c4);
                n0 = fmaf(a0.x, xv.x, fmaf(a0.y, xv.y, fmaf(a0.z, xv.z, fmaf(a0.w, xv.w, n0))));
                n0 = fmaf(b0.x, uv.x, fmaf(b0.y, uv.y, fmaf(b0.z, uv.z, fmaf(b0.w, uv.w, n0))));
                n1 = fmaf(a1.x, xv.x, fmaf(a1.y, xv.y, fmaf(a1.z, xv.z, fmaf(a1.w, xv.w, n1))));
                n1 = fmaf(b1.x, uv.x, fmaf(b1.y, uv.y, fmaf(b1.z, uv.z, fmaf(b1.w, uv.w, n1))));
            }
            __syncwarp();                                     // x_t and u_t consumed
            xs[lane] = n0;
            xs[lane + 32] = n1;
            if (xo) {
                store_out(p.x, xoff + (long long)(ts + 1) * N + lane, n0, obf);
                store_out(p.x, xoff + (long long)(ts + 1) * N + lane + 32, n1, obf);
            }
            __syncwarp();
        }
    }
}
inline size_t rollout_smem_bytes() { return sizeof(RollSmem); }

// Exercises the give-up branch of mbar_wait without any MMA in flight: one warp initialises a barrier on which
// nothing ever arrives, polls it `limit` times, and reports through the same kind of error word as the solver.
// The kernel returns by itself after `limit` polls.
__global__ void bounded_wait_selftest_kernel(int limit, int* error_flag)
{
    __shared__ unsigned long long bar;
    const uint32_t mbar = smem_u32(&bar);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(mbar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0 && !mbar_wait(mbar, 0u, limit))
        atomicExch(error_flag, 1);
}

inline size_t smem_bytes() { return SMEM_BYTES; }

} // namespace umma64
} // namespace ttc
