// Riccati-backward kernel for n = m = 64 when only P_0 and u_0 are wanted (tcgen05.mma, kind::tf32, accumulators in
// tensor memory).  Same organisation and the same five contractions per step as riccati_umma64_kernel (one persistent
// CTA per SM, four independent warpgroups, one instance per warpgroup, the tall matrix [S; Y'] factored in tensor
// memory), with a SHORTER DEPENDENCY CHAIN per step:
//
//   * 16-wide panels, factored in two levels.  The warp that owns the 16 diagonal rows factors the leading 8 x 8
//     block, forward-substitutes its own rows, exchanges the 8 x 8 block L21 through shared memory (warp-level
//     synchronisation only), updates and factors the second 8 x 8 block, and publishes L11, L21, L22.  After ONE
//     warpgroup barrier every thread applies the whole 16 x 16 triangular solve to its row in registers, and ONE
//     rank-16 trailing update (2 k-steps x 3 tf32 passes) goes to the tensor core.  A step has 4 panel round trips
//     (publish -> barrier -> substitute -> fence -> barrier -> MMA -> completion wait -> tcgen05.ld) instead of 8.
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
    alignas(16) float dg[2][64]; // the two 8 x 8 diagonal blocks of the current panel (rows of 8)
    alignas(16) float l21[64];   // rows of L21 = G21 L11^{-T}
    alignas(16) float ld[2][36]; // L11 and L22: strict lower triangle (28) + reciprocal pivots (8)
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
// strict lower triangle + reciprocal pivots of an 8 x 8 factor <-> 9 16-byte words
__device__ __forceinline__ void pack_factor(float* dst36, const float (&l)[8][8], const float (&rinv)[8])
{
    float4* d = reinterpret_cast<float4*>(dst36);
    d[0] = make_float4(l[1][0], l[2][0], l[2][1], l[3][0]);
    d[1] = make_float4(l[3][1], l[3][2], l[4][0], l[4][1]);
    d[2] = make_float4(l[4][2], l[4][3], l[5][0], l[5][1]);
    d[3] = make_float4(l[5][2], l[5][3], l[5][4], l[6][0]);
    d[4] = make_float4(l[6][1], l[6][2], l[6][3], l[6][4]);
    d[5] = make_float4(l[6][5], l[7][0], l[7][1], l[7][2]);
    d[6] = make_float4(l[7][3], l[7][4], l[7][5], l[7][6]);
    d[7] = make_float4(rinv[0], rinv[1], rinv[2], rinv[3]);
    d[8] = make_float4(rinv[4], rinv[5], rinv[6], rinv[7]);
}
__device__ __forceinline__ void unpack_factor(float (&l)[8][8], float (&rinv)[8], const float* src36)
{
    const float4* s = reinterpret_cast<const float4*>(src36);
    const float4 c0 = s[0], c1 = s[1], c2 = s[2], c3 = s[3], c4 = s[4], c5 = s[5], c6 = s[6], c7 = s[7], c8 = s[8];
    l[1][0] = c0.x; l[2][0] = c0.y; l[2][1] = c0.z; l[3][0] = c0.w;
    l[3][1] = c1.x; l[3][2] = c1.y; l[4][0] = c1.z; l[4][1] = c1.w;
    l[4][2] = c2.x; l[4][3] = c2.y; l[5][0] = c2.z; l[5][1] = c2.w;
    l[5][2] = c3.x; l[5][3] = c3.y; l[5][4] = c3.z; l[6][0] = c3.w;
    l[6][1] = c4.x; l[6][2] = c4.y; l[6][3] = c4.z; l[6][4] = c4.w;
    l[6][5] = c5.x; l[7][0] = c5.y; l[7][1] = c5.z; l[7][2] = c5.w;
    l[7][3] = c6.x; l[7][4] = c6.y; l[7][5] = c6.z; l[7][6] = c6.w;
    rinv[0] = c7.x; rinv[1] = c7.y; rinv[2] = c7.z; rinv[3] = c7.w;
    rinv[4] = c8.x; rinv[5] = c8.y; rinv[6] = c8.z; rinv[7] = c8.w;
}
__device__ __forceinline__ void load_block8(float (&l)[8][8], const float* blk)
{
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float4 a4 = *reinterpret_cast<const float4*>(blk + 8 * i);
        const float4 b4 = *reinterpret_cast<const float4*>(blk + 8 * i + 4);
        l[i][0] = a4.x; l[i][1] = a4.y; l[i][2] = a4.z; l[i][3] = a4.w;
        l[i][4] = b4.x; l[i][5] = b4.y; l[i][6] = b4.z; l[i][7] = b4.w;
    }
}
// hi[j] -= sum_k lo[k] * L21[j][k]  (the row's columns 8..15 after the first 8 have been substituted)
__device__ __forceinline__ void schur_row8(float (&hi)[8], const float (&lo)[8], const float* l21)
{
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float4 a4 = *reinterpret_cast<const float4*>(l21 + 8 * j);
        const float4 b4 = *reinterpret_cast<const float4*>(l21 + 8 * j + 4);
        float acc = hi[j];
        acc = fmaf(-lo[0], a4.x, acc); acc = fmaf(-lo[1], a4.y, acc); acc = fmaf(-lo[2], a4.z, acc); acc = fmaf(-lo[3], a4.w, acc);
        acc = fmaf(-lo[4], b4.x, acc); acc = fmaf(-lo[5], b4.y, acc); acc = fmaf(-lo[6], b4.z, acc); acc = fmaf(-lo[7], b4.w, acc);
        hi[j] = acc;
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
                float vlo[8], vhi[8];                          // the row's 16 panel columns
                auto load_cols = [&](int c0) {
                    uint32_t raw[16];
                    tmem_ld16(RF + lane_sel + c0, raw);
                    float4 r0 = make_float4(0.f, 0.f, 0.f, 0.f), r1 = r0, r2 = r0, r3 = r0;
                    if (warp < 2) {
                        const float4* rr = reinterpret_cast<const float4*>(Rs + wt * R_LD + c0);
                        r0 = rr[0]; r1 = rr[1]; r2 = rr[2]; r3 = rr[3];
                    }
                    tmem_wait_ld();
                    vlo[0] = __uint_as_float(raw[0]) + r0.x; vlo[1] = __uint_as_float(raw[1]) + r0.y;
                    vlo[2] = __uint_as_float(raw[2]) + r0.z; vlo[3] = __uint_as_float(raw[3]) + r0.w;
                    vlo[4] = __uint_as_float(raw[4]) + r1.x; vlo[5] = __uint_as_float(raw[5]) + r1.y;
                    vlo[6] = __uint_as_float(raw[6]) + r1.z; vlo[7] = __uint_as_float(raw[7]) + r1.w;
                    vhi[0] = __uint_as_float(raw[8]) + r2.x; vhi[1] = __uint_as_float(raw[9]) + r2.y;
                    vhi[2] = __uint_as_float(raw[10]) + r2.z; vhi[3] = __uint_as_float(raw[11]) + r2.w;
                    vhi[4] = __uint_as_float(raw[12]) + r3.x; vhi[5] = __uint_as_float(raw[13]) + r3.y;
                    vhi[6] = __uint_as_float(raw[14]) + r3.z; vhi[7] = __uint_as_float(raw[15]) + r3.w;
                };
                load_cols(0);
#pragma unroll 1
                for (int pnl = 0; pnl < NPANEL; ++pnl) {
                    const int col = PW * pnl;
                    const bool diag_warp = warp == (pnl >> 1);
                    if (diag_warp) {
                        // The 16 diagonal rows belong to this warp.  Two-level factorisation of the 16 x 16 block with
                        // warp-level synchronisation only; every lane of the warp substitutes its own row on the way.
                        const int r16 = wt - col;                               // 0..15 for the owners of the block rows
                        if ((unsigned)r16 < 8u) {
                            float4* dst = reinterpret_cast<float4*>(&misc.dg[0][8 * r16]);
                            dst[0] = make_float4(vlo[0], vlo[1], vlo[2], vlo[3]);
                            dst[1] = make_float4(vlo[4], vlo[5], vlo[6], vlo[7]);
                        }
                        __syncwarp();
                        int bad;
                        {
                            float l[8][8], rinv[8];
                            load_block8(l, &misc.dg[0][0]);
                            bad = chol8(l, rinv);
                            if (lane == 0)
                                pack_factor(&misc.ld[0][0], l, rinv);
                            fsub8(vlo, l, rinv);
                        }
                        if ((unsigned)(r16 - 8) < 8u) {                         // rows of L21
                            float4* dst = reinterpret_cast<float4*>(&misc.l21[8 * (r16 - 8)]);
                            dst[0] = make_float4(vlo[0], vlo[1], vlo[2], vlo[3]);
                            dst[1] = make_float4(vlo[4], vlo[5], vlo[6], vlo[7]);
                        }
                        __syncwarp();
                        schur_row8(vhi, vlo, &misc.l21[0]);
                        if ((unsigned)(r16 - 8) < 8u) {
                            float4* dst = reinterpret_cast<float4*>(&misc.dg[1][8 * (r16 - 8)]);
                            dst[0] = make_float4(vhi[0], vhi[1], vhi[2], vhi[3]);
                            dst[1] = make_float4(vhi[4], vhi[5], vhi[6], vhi[7]);
                        }
                        __syncwarp();
                        {
                            float l[8][8], rinv[8];
                            load_block8(l, &misc.dg[1][0]);
                            const int bad2 = chol8(l, rinv);
                            if (!bad && bad2)
                                bad = 8 + bad2;
                            if (lane == 0) {
                                pack_factor(&misc.ld[1][0], l, rinv);
                                if (bad && misc.flag == 0)
                                    misc.flag = ts * N + col + bad;
                            }
                            fsub8(vhi, l, rinv);
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
                    if (!diag_warp) {
                        {
                            float l[8][8], rinv[8];
                            unpack_factor(l, rinv, &misc.ld[0][0]);
                            fsub8(vlo, l, rinv);
                        }
                        schur_row8(vhi, vlo, &misc.l21[0]);
                        {
                            float l[8][8], rinv[8];
                            unpack_factor(l, rinv, &misc.ld[1][0]);
                            fsub8(vhi, l, rinv);
                        }
                    }
                    {
                        unsigned char* ph = PH + (uint32_t)(wt >> 3) * PSR16 + (uint32_t)(wt & 7) * 16u;
                        float h[16];
                        if (warp < 2) {                        // row wt of L: lower triangular, ends at column wt
                            float lo[16];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                if (col + j > wt)
                                    vlo[j] = 0.f;
                                if (col + 8 + j > wt)
                                    vhi[j] = 0.f;
                                h[j] = round_tf32(vlo[j]);
                                lo[j] = vlo[j] - h[j];
                                h[8 + j] = round_tf32(vhi[j]);
                                lo[8 + j] = vhi[j] - h[8 + j];
                            }
                            unsigned char* pl = PL + (uint32_t)(wt >> 3) * PSR16 + (uint32_t)(wt & 7) * 16u;
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4)
                                *reinterpret_cast<float4*>(pl + q4 * SC) = make_float4(lo[4 * q4], lo[4 * q4 + 1], lo[4 * q4 + 2], lo[4 * q4 + 3]);
                            if (keep_l) {                      // fp32 copy for u_0, packed by rows
                                float* row = Lp + lp_row(wt) + col;
                                if (col <= wt)
                                    *reinterpret_cast<float4*>(row) = make_float4(vlo[0], vlo[1], vlo[2], vlo[3]);
                                if (col + 4 <= wt)
                                    *reinterpret_cast<float4*>(row + 4) = make_float4(vlo[4], vlo[5], vlo[6], vlo[7]);
                                if (col + 8 <= wt)
                                    *reinterpret_cast<float4*>(row + 8) = make_float4(vhi[0], vhi[1], vhi[2], vhi[3]);
                                if (col + 12 <= wt)
                                    *reinterpret_cast<float4*>(row + 12) = make_float4(vhi[4], vhi[5], vhi[6], vhi[7]);
                            }
                        } else {                               // row wt - 64 of Z': kept as tf32 (operand of (5)), low part zero
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                h[j] = round_tf32(vlo[j]);
                                h[8 + j] = round_tf32(vhi[j]);
                            }
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
