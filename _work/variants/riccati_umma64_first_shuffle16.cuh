// Riccati-backward kernel for n = m = 64 when only P_0 and u_0 are wanted (tcgen05.mma, kind::tf32, accumulators in
// tensor memory).  Same organisation and the same five contractions per step as riccati_umma64_kernel (one persistent
// CTA per SM, four independent warpgroups, one instance per warpgroup, the tall matrix [S; Y'] factored in tensor
// memory), with a SHORTER DEPENDENCY CHAIN per step:
//
//   * 16-wide panels.  The 16 lanes that own the diagonal rows factor the 16 x 16 block among themselves with
//     shuffles (one row per lane, straight from the registers the tensor-memory load filled: no gather through
//     shared memory) and publish the factor; after ONE warpgroup barrier every other thread applies the 16 x 16
//     triangular solve to its row in registers, and ONE rank-16 trailing update (2 k-steps x 3 tf32 passes) goes to
//     the tensor core.  A step has 4 panel round trips (publish -> barrier -> substitute -> fence -> barrier ->
//     MMA -> completion wait -> tcgen05.ld) instead of 8.
//   * The fp32 factor L is kept only at the last step (u_0 needs it), packed by rows, so the second 64 x 64 buffer
//     of the general kernel is gone and the wider panel buffers fit.
//   * The rows of Q for the read-out P_t = Q + A'P A - Z'Z are fetched into registers while the last contraction
//     is in flight.
//
// Per step (Prop. 3.1), with P symmetric:
//   (1) W = BA P -> [V'; T']          SS, M128 N64          (2) F = W B = [S - R; Y']      TS
//   (3) [S; Y'] = [L; Z'] L'          blocked, in tensor memory, 16-wide panels
//   (4) DP = W A                      TS, into the columns of F          (5) DP -= Z' Z      SS
//   P <- Q + DP ; at the last step u_0 = -L^{-T} (Z x_0)
#pragma once

#include "riccati_umma64.cuh"

namespace ttc {
namespace umma64 {
namespace first {

constexpr int PW = 16;                          // panel width
constexpr int NPANEL = N / PW;
constexpr uint32_t PSR16 = 512;                 // bytes between 8-row groups of a 128 x 16 panel buffer (4 chunks)
constexpr uint32_t PAN16_BYTES = 16 * PSR16;    // one 128 x 16 buffer
constexpr int LP_FLOATS = 2176;                 // packed lower triangle, rows padded to a multiple of 4 columns

// first float of row r of the packed factor: rows 4q .. 4q + 3 hold 4 (q + 1) floats each
__device__ __forceinline__ int lp_row(int r)
{
    const int q = r >> 2, s = r & 3;
    return 4 * (q + 1) * (2 * q + s);
}

constexpr uint32_t OFF_X0 = 0;
constexpr uint32_t OFF_PH = MAT_BYTES;
constexpr uint32_t OFF_PL = MAT_BYTES + PAN16_BYTES;
constexpr uint32_t OFF_LP = MAT_BYTES + 2 * PAN16_BYTES;
constexpr uint32_t OFF_MISC = OFF_LP + LP_FLOATS * 4;
struct Misc {
    unsigned long long mbar;     // MMA completion barrier (every thread waits on it)
    unsigned long long mbar_w;   // completion of W = BA P: only the issuing thread waits on it
    int dead;                    // set when a wait timed out
    int flag;                    // first failed pivot (0 = none)
    alignas(16) float x0[N];
    alignas(16) float y0[N];     // Z x_0, then the back substitution's running right-hand side
    alignas(16) float lpub[160]; // factor of the current 16 x 16 diagonal block as published to the warpgroup
};
constexpr uint32_t WG_BYTES = OFF_MISC + ((sizeof(Misc) + 127) / 128) * 128;
constexpr uint32_t SMEM_BYTES = BUF_BYTES + R_BYTES + NUM_WG * WG_BYTES + 128;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
static_assert(OFF_LP % 16 == 0 && OFF_MISC % 16 == 0, "16-byte rows");

__device__ __forceinline__ uint64_t panel16_desc(uint32_t saddr)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)(SC >> 4) << 16) | ((uint64_t)(PSR16 >> 4) << 32) |
           ((uint64_t)1 << 46);
}
// 32 lanes x 16 consecutive columns; the caller waits with tmem_wait_ld() before it reads r
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
}
// Cholesky of a 16 x 16 SPD block spread over a 16-lane segment (lane i of the segment = row i), right-looking with
// shuffles: pivot j is broadcast from lane j, every lane scales its entry of column j and updates the columns right of
// it with the entries of the rows below, which arrive by shuffle.  The chain from one pivot to the next is
// shuffle -> reciprocal -> multiply -> fma.  On return s[0..i] is row i of L (entries right of the diagonal are
// meaningless) and rs_own = 1 / L[i][i].  Returns 0 or 1 + the index of the first non-positive pivot (uniform).
__device__ __forceinline__ int seg_chol16(float (&s)[16], float& rs_own, int i)
{
    int bad = 0;
    rs_own = 1.f;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const float sj = s[j];
        float d = __shfl_sync(0xffffffffu, sj, j, 16);
        if (!(d > 0.f)) {
            if (!bad)
                bad = j + 1;
            d = 1.f;
        }
        float rs;
        asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(rs) : "f"(d));
        const float f = sj * rs * rs;                          // s_ij / d_j
#pragma unroll
        for (int cc = j + 1; cc < 16; ++cc) {
            const float lc = __shfl_sync(0xffffffffu, sj, cc, 16);
            s[cc] = fmaf(-f, lc, s[cc]);
        }
        s[j] = sj * rs;
        if (i == j)
            rs_own = rs;
    }
    return bad;
}
// Published form of the 16 x 16 factor: the strict lower triangle with row i (i >= 1) padded to a multiple of four
// floats, rows in order (144 floats), then the 16 reciprocal pivots: 40 16-byte words.
constexpr int LPUB_FLOATS = 160;
__host__ __device__ constexpr int lpub_row(int i)              // first float of row i >= 1
{
    return 8 * ((i - 1) >> 2) * (((i - 1) >> 2) + 1) + ((i - 1) & 3) * 4 * (((i - 1) >> 2) + 1);
}
// x (a row of 16) <- x L^{-T} with the published factor
__device__ __forceinline__ void fsub16(float (&x)[16], const float* lpub)
{
    float rinv[16];
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
        const float4 r4 = *reinterpret_cast<const float4*>(lpub + 144 + 4 * q4);
        rinv[4 * q4] = r4.x; rinv[4 * q4 + 1] = r4.y; rinv[4 * q4 + 2] = r4.z; rinv[4 * q4 + 3] = r4.w;
    }
    x[0] *= rinv[0];
#pragma unroll
    for (int i = 1; i < 16; ++i) {
        float acc = x[i];
#pragma unroll
        for (int q4 = 0; q4 <= (i - 1) >> 2; ++q4) {
            const float4 l4 = *reinterpret_cast<const float4*>(lpub + lpub_row(i) + 4 * q4);
            if (4 * q4 + 0 < i) acc = fmaf(-l4.x, x[4 * q4 + 0], acc);
            if (4 * q4 + 1 < i) acc = fmaf(-l4.y, x[4 * q4 + 1], acc);
            if (4 * q4 + 2 < i) acc = fmaf(-l4.z, x[4 * q4 + 2], acc);
            if (4 * q4 + 3 < i) acc = fmaf(-l4.w, x[4 * q4 + 3], acc);
        }
        x[i] = acc * rinv[i];
    }
}

__global__ void __launch_bounds__(THREADS, 1) riccati_umma64_first_kernel(SolveParams p, int* chunk_counter, int* error_flag)
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
    unsigned char* X0 = wsm + OFF_X0;        // P -> Z' -> next P
    unsigned char* PH = wsm + OFF_PH;        // panel operand, hi parts (128 x 16)
    unsigned char* PL = wsm + OFF_PL;        // panel operand, lo parts
    float* Lp = reinterpret_cast<float*>(wsm + OFF_LP);          // fp32 L of the last step, packed by rows
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
    auto zero_pl_tail = [&]() {
        if (wt >= 64)
            for (int e = wt - 64; e < 256; e += 64)
                *reinterpret_cast<float4*>(PL + 8u * PSR16 + (uint32_t)e * 16u) = make_float4(0.f, 0.f, 0.f, 0.f);
    };
    zero_pl_tail();
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
    const bool want_u0 = p.u != nullptr;
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
                    // F reads W from tensor memory: an MMA whose A operand was written by the MMAs just before it is
                    // not ordered after them by the pipe, so the issuing thread waits for W on a barrier of its own
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
                // (3) [S; Y'] = [L; Z'] L', 16 columns at a time; thread wt owns row wt
                const bool keep_l = ts == 0 && want_u0;
                float v[16];                                   // the row's 16 panel columns
                auto load_cols = [&](int c0) {
                    uint32_t raw[16];
                    tmem_ld16(RF + lane_sel + c0, raw);
                    float4 r0 = make_float4(0.f, 0.f, 0.f, 0.f), r1 = r0, r2 = r0, r3 = r0;
                    if (warp < 2) {
                        const float4* rr = reinterpret_cast<const float4*>(Rs + wt * R_LD + c0);
                        r0 = rr[0]; r1 = rr[1]; r2 = rr[2]; r3 = rr[3];
                    }
                    tmem_wait_ld();
                    v[0] = __uint_as_float(raw[0]) + r0.x; v[1] = __uint_as_float(raw[1]) + r0.y;
                    v[2] = __uint_as_float(raw[2]) + r0.z; v[3] = __uint_as_float(raw[3]) + r0.w;
                    v[4] = __uint_as_float(raw[4]) + r1.x; v[5] = __uint_as_float(raw[5]) + r1.y;
                    v[6] = __uint_as_float(raw[6]) + r1.z; v[7] = __uint_as_float(raw[7]) + r1.w;
                    v[8] = __uint_as_float(raw[8]) + r2.x; v[9] = __uint_as_float(raw[9]) + r2.y;
                    v[10] = __uint_as_float(raw[10]) + r2.z; v[11] = __uint_as_float(raw[11]) + r2.w;
                    v[12] = __uint_as_float(raw[12]) + r3.x; v[13] = __uint_as_float(raw[13]) + r3.y;
                    v[14] = __uint_as_float(raw[14]) + r3.z; v[15] = __uint_as_float(raw[15]) + r3.w;
                };
                load_cols(0);
#pragma unroll 1
                for (int pnl = 0; pnl < NPANEL; ++pnl) {
                    const int col = PW * pnl;
                    const bool diag_warp = warp == (pnl >> 1);
                    bool owner = false;                        // this thread owns one of the 16 diagonal rows
                    if (diag_warp) {
                        // The 16 diagonal rows are one 16-lane segment of this warp: factor the block with shuffles
                        // (the other segment runs the same instructions on its own rows and discards the result).
                        float sblk[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            sblk[j] = v[j];
                        const int i = lane & 15;
                        float rs_own;
                        const int bad = seg_chol16(sblk, rs_own, i);
                        owner = (lane >> 4) == (pnl & 1);
                        if (owner) {
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                v[j] = sblk[j];                // row i of L (masked right of the diagonal below)
                            misc.lpub[144 + i] = rs_own;
                            if (i >= 1) {
                                float* dst = &misc.lpub[lpub_row(i)];
#pragma unroll
                                for (int q4 = 0; q4 < 4; ++q4)
                                    if (4 * q4 < i)
                                        *reinterpret_cast<float4*>(dst + 4 * q4) = make_float4(sblk[4 * q4], sblk[4 * q4 + 1], sblk[4 * q4 + 2], sblk[4 * q4 + 3]);
                            }
                            if (bad && i == 0 && misc.flag == 0)
                                misc.flag = ts * N + col + bad;
                        }
                    }
                    tc_fence_before();
                    wg_barrier(wg);
                    if (misc.dead != 0) {
                        dead = true;
                        break;
                    }
                    if (pnl == NPANEL - 1 && issuer) {
                        // every row has read its last columns of F: (4) DP = W A into the columns of F
                        tc_fence_after();
                        gemm_ts(RF, RW, smem_u32(BA) + MAT_BYTES, 64);
                    }
                    if (!owner)
                        fsub16(v, &misc.lpub[0]);
                    {
                        unsigned char* ph = PH + (uint32_t)(wt >> 3) * PSR16 + (uint32_t)(wt & 7) * 16u;
                        float h[16];
                        if (warp < 2) {                        // row wt of L: lower triangular, ends at column wt
                            float lo[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                if (col + j > wt)
                                    v[j] = 0.f;
                                h[j] = round_tf32(v[j]);
                                lo[j] = v[j] - h[j];
                            }
                            unsigned char* pl = PL + (uint32_t)(wt >> 3) * PSR16 + (uint32_t)(wt & 7) * 16u;
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4)
                                *reinterpret_cast<float4*>(pl + q4 * SC) = make_float4(lo[4 * q4], lo[4 * q4 + 1], lo[4 * q4 + 2], lo[4 * q4 + 3]);
                            if (keep_l) {                      // fp32 copy for u_0, packed by rows
                                float* row = Lp + lp_row(wt) + col;
#pragma unroll
                                for (int q4 = 0; q4 < 4; ++q4)
                                    if (col + 4 * q4 <= wt)
                                        *reinterpret_cast<float4*>(row + 4 * q4) = make_float4(v[4 * q4], v[4 * q4 + 1], v[4 * q4 + 2], v[4 * q4 + 3]);
                            }
                        } else {                               // row wt - 64 of Z': kept as tf32 (operand of (5)), low part zero
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                h[j] = round_tf32(v[j]);
                            unsigned char* pz = X0 + (uint32_t)((wt - 64) >> 3) * SR + 4u * pnl * SC + (uint32_t)(wt & 7) * 16u;
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4)
                                *reinterpret_cast<float4*>(pz + q4 * SC) = make_float4(h[4 * q4], h[4 * q4 + 1], h[4 * q4 + 2], h[4 * q4 + 3]);
                        }
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4)
                            *reinterpret_cast<float4*>(ph + q4 * SC) = make_float4(h[4 * q4], h[4 * q4 + 1], h[4 * q4 + 2], h[4 * q4 + 3]);
                    }
                    if (pnl == NPANEL - 1)
                        break;
                    async_proxy_fence();
                    wg_barrier(wg);
                    if (issuer) {                              // G -= panel * panel[0:64]'  (hi*hi + lo*hi + hi*lo), K = 16
                        tc_fence_after();
                        const uint32_t idn = instr_desc(64, 1);
#pragma unroll
                        for (int k2 = 0; k2 < 2; ++k2) {
                            const uint64_t dh = panel16_desc(smem_u32(PH) + 2u * k2 * SC), dl = panel16_desc(smem_u32(PL) + 2u * k2 * SC);
                            mma_ss(RF, dh, dh, idn, 1u);
                            mma_ss(RF, dl, dh, idn, 1u);
                            mma_ss(RF, dh, dl, idn, 1u);
                        }
                        mma_commit(mbar);
                    }
                    wait_mma();
                    load_cols(col + PW);
                }
                async_proxy_fence();
                tc_fence_before();
                wg_barrier(wg);
                dead = dead || misc.dead != 0;
                // (5) DP -= Z' Z : A operand rows 64..127 = Z'; rows 0..63 are whatever precedes X0 in shared memory
                // (they feed accumulator lanes that are never read)
                if (issuer && !dead) {
                    tc_fence_after();
                    gemm_ss(RF, smem_u32(X0) - MAT_BYTES, smem_u32(X0), 64, 1, true);
                    mma_commit(mbar);
                }
                if (dead)
                    break;
                // the rows of Q for the read-out travel while (5) is in flight (bf16: the whole row in 32 registers)
                uint4 qraw[8];
                const bool q_bf16 = p.Q.dtype == TTC_BF16;
                if (warp >= 2 && q_bf16) {
                    const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.Q.ptr) + oq + (long long)(wt - 64) * N);
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        qraw[c] = __ldg(src + c);
                }
                if (keep_l && warp < 2) {
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
                        float w[8];
#pragma unroll
                        for (int r = 0; r < 8; ++r)
                            w[r] = misc.y0[c0 + r];
#pragma unroll
                        for (int r = 7; r >= 0; --r) {
                            float vv = w[r];
#pragma unroll
                            for (int j = r + 1; j < 8; ++j)
                                vv = fmaf(-Lp[lp_row(c0 + j) + c0 + r], w[j], vv);
                            w[r] = vv / Lp[lp_row(c0 + r) + c0 + r];
                        }
                        if (i < c0) {
#pragma unroll
                            for (int r = 0; r < 8; ++r)
                                zi = fmaf(-Lp[lp_row(c0 + r) + i], w[r], zi);
                        }
                        half_barrier(wg);
                        if (i < c0)
                            misc.y0[i] = zi;
#pragma unroll
                        for (int r = 0; r < 8; ++r)
                            if (i == c0 + r)
                                p.u[inst * (long long)N + i] = -w[r];
                    }
                }
                wait_mma();
                // P_t = Q + DP: warps 2, 3 own the rows (lanes 64..127)
                if (warp >= 2) {
                    const int j = wt - 64;
#pragma unroll
                    for (int qt = 0; qt < 4; ++qt) {           // 16 columns at a time
                        float q[16];
                        if (q_bf16) {
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
                        } else {
                            const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.Q.ptr) + oq + (long long)j * N + 16 * qt);
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const float4 v4 = __ldg(src + c);
                                q[4 * c] = v4.x; q[4 * c + 1] = v4.y; q[4 * c + 2] = v4.z; q[4 * c + 3] = v4.w;
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
                        } else if (p.P) {
                            float4* dst = reinterpret_cast<float4*>(p.P + inst * (long long)N * N + (long long)j * N + 16 * qt);
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                dst[c] = make_float4(q[4 * c], q[4 * c + 1], q[4 * c + 2], q[4 * c + 3]);
                        }
                    }
                    // Every eighth step the operand is replaced by (P + P') / 2: Q and Z'Z are symmetric but the rounding
                    // of A'(P A) is not, and the antisymmetric part E obeys E <- A'E A, which grows along an open-loop
                    // unstable A however well the closed loop is damped.  The two panel buffers (16 KB, contiguous, idle
                    // here) take the averaged rows; the zero tail of the low-part buffer is restored afterwards.
                    if (ts > 0 && (ts & 7) == 0) {
                        half_barrier(wg);                     // both halves of every row are in X0
#pragma unroll 8
                        for (int c = 0; c < 64; ++c) {
                            const int cj = (c + (j >> 2)) & 63;       // rotated per lane: the column reads hit 32 banks
                            elem(PH, toff(j, cj)) = round_tf32(0.5f * (elem(X0, toff(j, cj)) + elem(X0, toff(cj, j))));
                        }
                        half_barrier(wg);                     // every column has been read
#pragma unroll
                        for (int c = 0; c < 16; ++c)
                            *reinterpret_cast<float4*>(X0 + toff(j, 4 * c)) = *reinterpret_cast<const float4*>(PH + toff(j, 4 * c));
                        half_barrier(wg);                     // every row has been copied back
                        zero_pl_tail();
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
                if (fl)
                    wg_fail_instance(p, inst, fl, wt);
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

inline size_t smem_bytes() { return SMEM_BYTES; }

} // namespace first
} // namespace umma64
} // namespace ttc
