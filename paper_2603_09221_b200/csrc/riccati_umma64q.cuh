// Riccati-backward kernel for n = m = 64 on the tcgen05 tensor cores, four warpgroups per CTA.
//
// Same step as riccati_umma64_kernel (Prop. 3.1; see that file for the formulas and the operand layout), arranged
// for more independent dependency chains per SM: every warpgroup (128 threads = the 128 lanes of tensor memory) walks
// ONE instance through the horizon, four warpgroups share the per-head operand BA = [B'; A'], and a thread gets 128
// registers.  The step is one long chain (64 pivots in 8 panels, each panel a tensor-memory load, an 8 x 8 Cholesky,
// a broadcast, a row update, an operand store and a tcgen05 round trip); four shorter chains keep the SM busier than
// two chains that each carry a pair of instances.
//
// Per warpgroup: tensor memory columns R_W (W = BA P') and R_F (F = W B = [S - R; Y'], later DP = W A - Z'Z);
// shared memory X1 (L in fp32, only when the gains or u_0 need it) | X0 (P, then Z') | panel hi | panel lo | scratch.
// X1 directly precedes X0: step (5) starts its A operand 64 rows before Z' so that Z' lands on lanes 64..127.
#pragma once

#include "riccati_umma64.cuh"

namespace ttc {
namespace umma64 {

constexpr int NUM_WG4 = 4;
constexpr int THREADS4 = NUM_WG4 * WG_THREADS;
constexpr int TOK4 = 8;                                  // tokens per warpgroup and work item
constexpr int CHUNK4 = NUM_WG4 * TOK4;                   // tokens per work item of a CTA
constexpr uint32_t Q_OFF_X1 = 0;
constexpr uint32_t Q_OFF_X0 = MAT_BYTES;
constexpr uint32_t Q_OFF_PH = 2 * MAT_BYTES;
constexpr uint32_t Q_OFF_PL = 2 * MAT_BYTES + PAN_BYTES;
constexpr uint32_t Q_OFF_MISC = 2 * MAT_BYTES + 2 * PAN_BYTES;
struct Misc4 {
    unsigned long long mbar;     // MMA completion barrier (every thread waits on it)
    unsigned long long mbar_w;   // completion of W = BA P': only the issuing thread waits on it
    int dead;                    // set when a wait timed out
    int flag;                    // first failed pivot (0 = none)
    alignas(16) float x0[N];
    alignas(16) float y0[N];     // Y x_0 / u_t of the rollout; during the factorisation: the 8 x 8 diagonal block
    alignas(16) float ld[36];    // current diagonal factor: strict lower triangle (28) + reciprocal pivots (8)
};
constexpr uint32_t WG4_BYTES = Q_OFF_MISC + ((sizeof(Misc4) + 127) / 128) * 128;
struct Cta4 {
    int chunk;                   // current work item
    int dead;                    // some warpgroup gave up: the CTA stops taking work
    uint32_t tmem_base;
};
constexpr uint32_t SMEM4_BYTES = BUF_BYTES + NUM_WG4 * WG4_BYTES + 128;
static_assert(SMEM4_BYTES <= 227 * 1024, "shared memory of one CTA");

__device__ __forceinline__ void wg_barrier4(int wg) { asm volatile("bar.sync %0, %1;" :: "r"(10 + wg), "r"(WG_THREADS) : "memory"); }

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
__device__ __forceinline__ void store_half_global(float* dst, const float (&v)[32])
{
#pragma unroll
    for (int c = 0; c < 8; ++c)
        reinterpret_cast<float4*>(dst)[c] = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
}

// GAINS = the request needs every K_t (K, x or the full u wanted); the other instantiation carries none of that code.
template <bool GAINS>
__global__ void __launch_bounds__(THREADS4, 1) riccati_umma64q_kernel(SolveParams p, int* chunk_counter, int* error_flag)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const int tid = threadIdx.x;
    const int wg = tid / WG_THREADS;
    const int wt = tid % WG_THREADS;
    const int warp = wt >> 5;                  // warp in warpgroup: owns tensor-memory lanes 32 warp .. 32 warp + 31
    const int lane = wt & 31;
    unsigned char* BA = smem_raw;              // rows 0..63: B' (row j = column j of B), rows 64..127: A'; shared by the CTA
    unsigned char* wsm = smem_raw + BUF_BYTES + (size_t)wg * WG4_BYTES;
    unsigned char* X1 = wsm + Q_OFF_X1;        // L, fp32 (kept only when the gains or u_0 need it)
    unsigned char* X0 = wsm + Q_OFF_X0;        // P -> Z' -> next P
    unsigned char* PH = wsm + Q_OFF_PH;        // panel operand, hi parts (128 x 8)
    unsigned char* PL = wsm + Q_OFF_PL;        // panel operand, lo parts
    Misc4& misc = *reinterpret_cast<Misc4*>(wsm + Q_OFF_MISC);
    Cta4& cta = *reinterpret_cast<Cta4*>(smem_raw + BUF_BYTES + (size_t)NUM_WG4 * WG4_BYTES);
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
    const long long chunks_per_head = (p.tcount + CHUNK4 - 1) / CHUNK4;
    const long long nchunks = p.b0 * p.b1 * chunks_per_head;
    constexpr bool need_K_all = GAINS;
    const bool want_u0 = (p.u != nullptr) && p.first_only && !need_K_all;
    const bool rollout = (p.x != nullptr) || (p.u != nullptr && need_K_all);
    float* Kbase = p.K ? p.K : p.Kws;
    long long offA_loaded = -1, offB_loaded = -1;
    const float* Rg = nullptr;
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
        const long long tok0 = p.t0 + (chunk % chunks_per_head) * CHUNK4;
        const long long inst0 = head * p.b2 + tok0;
        const int ntok = (int)min((long long)CHUNK4, p.t0 + p.tcount - tok0);
        {
            const long long oa = operand_offset(p.A, inst0, p.b1, p.b2);
            const long long ob = operand_offset(p.B, inst0, p.b1, p.b2);
            if (oa != offA_loaded || ob != offB_loaded) {
                const float* Ag = reinterpret_cast<const float*>(p.A.ptr) + oa;
                const float* Bg = reinterpret_cast<const float*>(p.B.ptr) + ob;
                for (int e = tid; e < N * N; e += THREADS4) {
                    const int k = e >> 6, j = e & 63;
                    elem(BA, toff(j, k)) = round_tf32(__ldg(Bg + e));
                    elem(BA, toff(64 + j, k)) = round_tf32(__ldg(Ag + e));
                }
                offA_loaded = oa; offB_loaded = ob;
                async_proxy_fence();
                __syncthreads();
            }
            Rg = reinterpret_cast<const float*>(p.R.ptr) + operand_offset(p.R, inst0, p.b1, p.b2);
        }
        const int my0 = TOK4 * wg, my1 = min(ntok, TOK4 * wg + TOK4);

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
                        store_half_global(p.P + (inst * (long long)(H + 1) + H) * N * N + (long long)j * N + 32 * half, q);
                }
            } else if (p.x0.ptr && warp == 0) {
                const long long ox = operand_offset(p.x0, inst, p.b1, p.b2);
                misc.x0[2 * lane] = load_elem(p.x0, ox + 2 * lane);
                misc.x0[2 * lane + 1] = load_elem(p.x0, ox + 2 * lane + 1);
            }
            if (wt == 0)
                misc.flag = 0;
            async_proxy_fence();
            wg_barrier4(wg);

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
                const bool keep_l = need_K_all || (ts == 0 && want_u0);
                float* diag = &misc.y0[0];                     // [8][8]
                float v[8];
                auto load_cols = [&](int c0) {
                    uint32_t raw[8];
                    tmem_ld8(RF + lane_sel + c0, raw);
                    float4 r0 = make_float4(0.f, 0.f, 0.f, 0.f), r1 = r0;
                    if (warp < 2) {
                        r0 = __ldg(reinterpret_cast<const float4*>(Rg + (long long)wt * N + c0));
                        r1 = __ldg(reinterpret_cast<const float4*>(Rg + (long long)wt * N + c0 + 4));
                    }
                    tmem_wait_ld();
                    v[0] = __uint_as_float(raw[0]) + r0.x; v[1] = __uint_as_float(raw[1]) + r0.y;
                    v[2] = __uint_as_float(raw[2]) + r0.z; v[3] = __uint_as_float(raw[3]) + r0.w;
                    v[4] = __uint_as_float(raw[4]) + r1.x; v[5] = __uint_as_float(raw[5]) + r1.y;
                    v[6] = __uint_as_float(raw[6]) + r1.z; v[7] = __uint_as_float(raw[7]) + r1.w;
                };
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
                    wg_barrier4(wg);
                    if (misc.dead != 0) {
                        dead = true;
                        break;
                    }
                    if (pnl == 7 && issuer) {
                        // every row has read its last columns of F: (4) DP = W A into the columns of F
                        tc_fence_after();
                        gemm_ts(RF, RW, smem_u32(BA) + MAT_BYTES, 64);
                    }
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
                    }
                    {
                        unsigned char* ph = PH + (uint32_t)(wt >> 3) * PSR + (uint32_t)(wt & 7) * 16u;
                        float hi[8];
                        if (warp < 2) {                        // row wt of L: lower triangular, ends at column wt
                            float lo[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                if (col + j > wt)
                                    v[j] = 0.f;
                                hi[j] = round_tf32(v[j]);
                                lo[j] = v[j] - hi[j];
                            }
                            unsigned char* pl = PL + (uint32_t)(wt >> 3) * PSR + (uint32_t)(wt & 7) * 16u;
                            *reinterpret_cast<float4*>(pl) = make_float4(lo[0], lo[1], lo[2], lo[3]);
                            *reinterpret_cast<float4*>(pl + SC) = make_float4(lo[4], lo[5], lo[6], lo[7]);
                            if (keep_l)                        // fp32 copy for the gains / u_0
                                store_row8<true, false>(X1 + (uint32_t)(wt >> 3) * SR + 2u * pnl * SC, wt & 7, v);
                        } else {                               // row wt - 64 of Z': kept as tf32 (operand of (5)), low part zero
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                hi[j] = round_tf32(v[j]);
                            unsigned char* pz = X0 + (uint32_t)((wt - 64) >> 3) * SR + 2u * pnl * SC + (uint32_t)(wt & 7) * 16u;
                            *reinterpret_cast<float4*>(pz) = make_float4(hi[0], hi[1], hi[2], hi[3]);
                            *reinterpret_cast<float4*>(pz + SC) = make_float4(hi[4], hi[5], hi[6], hi[7]);
                        }
                        *reinterpret_cast<float4*>(ph) = make_float4(hi[0], hi[1], hi[2], hi[3]);
                        *reinterpret_cast<float4*>(ph + SC) = make_float4(hi[4], hi[5], hi[6], hi[7]);
                    }
                    if (pnl == 7)
                        break;
                    async_proxy_fence();
                    wg_barrier4(wg);
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
                    load_cols(col + 8);
                }
                async_proxy_fence();
                tc_fence_before();
                wg_barrier4(wg);
                dead = dead || misc.dead != 0;
                // (5) DP -= Z' Z : A operand rows 64..127 = Z' (rows 0..63 = X1, unused lanes)
                if (issuer && !dead) {
                    tc_fence_after();
                    gemm_ss(RF, smem_u32(X0) - MAT_BYTES, smem_u32(X0), 64, 1, true);
                    mma_commit(mbar);
                }
                if (dead)
                    break;
                if (ts == 0 && want_u0 && warp < 2) {
                    // u_0 = K_0 x_0 = -L^{-T} (Z x_0), fp32, by the 64 threads of warps 0, 1
                    const int i = wt;
                    pair_barrier(wg, 0);
                    float zi = 0.f;
#pragma unroll 8
                    for (int c = 0; c < N; ++c)
                        zi = fmaf(elem(X0, toff(c, i)), misc.x0[c], zi);               // Z[i][c] = Z'[c][i]
                    misc.y0[i] = zi;
#pragma unroll 1
                    for (int kb = 7; kb >= 0; --kb) {           // back substitution L' w = Z x_0 in 8-wide blocks
                        pair_barrier(wg, 0);
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
                        pair_barrier(wg, 0);
                        if (i < c0)
                            misc.y0[i] = zi;
#pragma unroll
                        for (int r = 0; r < 8; ++r)
                            if (i == c0 + r)
                                p.u[inst * (long long)N + i] = -w[r];
                    }
                }
                wait_mma();
                if (need_K_all) {
                    // (5) has consumed Z': turn it into the gains in place, K_t[i][c] = -(Z' L^{-1})[c][i]
                    if (warp < 2) {
                        pair_gain_solve(X1, X0, wg, 0, warp, lane);
                        const int cidx = wt;
                        float* kt = Kbase + (inst * (long long)H + ts) * N * N + cidx;
                        const unsigned char* row = X0 + (uint32_t)(cidx >> 3) * SR + (uint32_t)(cidx & 7) * 16u;
#pragma unroll
                        for (int q4 = 0; q4 < 16; ++q4) {
                            const float4 kv = *reinterpret_cast<const float4*>(row + q4 * SC);
                            kt[(4 * q4 + 0) * N] = -kv.x;
                            kt[(4 * q4 + 1) * N] = -kv.y;
                            kt[(4 * q4 + 2) * N] = -kv.z;
                            kt[(4 * q4 + 3) * N] = -kv.w;
                        }
                    }
                    wg_barrier4(wg);                   // X0 is free for the next value matrix
                }
                // P_t = Q + DP: warps 2, 3 own the rows (lanes 64..127)
                if (warp >= 2) {
                    const int j = wt - 64;
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
                        if (p.P && (!p.first_only || ts == 0))
                            store_half_global(p.P + (inst * (long long)(p.first_only ? 1 : H + 1) + (p.first_only ? 0 : ts)) * N * N +
                                                  (long long)j * N + 32 * half, q);
                    }
                }
                tc_fence_before();
                async_proxy_fence();
                wg_barrier4(wg);
                dead = dead || misc.dead != 0;
            }
            if (dead)
                break;
            if (rollout && warp < 2) {
                // forward loop of Alg. 1 by 64 threads: u_t = K_t x_t, x_{t+1} = A x_t + B u_t (fp32)
                const int i = wt;
                const bool st = misc.flag == 0;
                float* xo = (p.x && st) ? p.x + inst * (long long)(H + 1) * N : nullptr;
                float* uo = (p.u && st) ? p.u + inst * (long long)(p.first_only ? 1 : H) * N : nullptr;
                const float4* Ar = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.A.ptr) + offA_loaded + (long long)i * N);
                const float4* Br = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.B.ptr) + offB_loaded + (long long)i * N);
                if (xo)
                    xo[i] = misc.x0[i];
#pragma unroll 1
                for (int ts = 0; ts < H; ++ts) {
                    const float4* kr = reinterpret_cast<const float4*>(Kbase + (inst * (long long)H + ts) * N * N + (long long)i * N);
                    float ui = 0.f;
#pragma unroll
                    for (int c4 = 0; c4 < 16; ++c4) {
                        const float4 kv = kr[c4];
                        const float4 xv = *reinterpret_cast<const float4*>(&misc.x0[4 * c4]);
                        ui = fmaf(kv.x, xv.x, fmaf(kv.y, xv.y, fmaf(kv.z, xv.z, fmaf(kv.w, xv.w, ui))));
                    }
                    misc.y0[i] = ui;
                    if (uo && (!p.first_only || ts == 0))
                        uo[(p.first_only ? 0 : (long long)ts * N) + i] = ui;
                    pair_barrier(wg, 0);
                    float xi = 0.f;
#pragma unroll
                    for (int c4 = 0; c4 < 16; ++c4) {
                        const float4 av = __ldg(Ar + c4), bv = __ldg(Br + c4);
                        const float4 xv = *reinterpret_cast<const float4*>(&misc.x0[4 * c4]);
                        const float4 uv = *reinterpret_cast<const float4*>(&misc.y0[4 * c4]);
                        xi = fmaf(av.x, xv.x, fmaf(av.y, xv.y, fmaf(av.z, xv.z, fmaf(av.w, xv.w, xi))));
                        xi = fmaf(bv.x, uv.x, fmaf(bv.y, uv.y, fmaf(bv.z, uv.z, fmaf(bv.w, uv.w, xi))));
                    }
                    pair_barrier(wg, 0);               // x_t and u_t consumed
                    misc.x0[i] = xi;
                    if (xo)
                        xo[(long long)(ts + 1) * N + i] = xi;
                    pair_barrier(wg, 0);
                }
            }
            wg_barrier4(wg);
            // ---- status / failed instance
            {
                const int fl = misc.flag;
                if (fl)
                    wg_fail_instance(p, inst, fl, wt);
                else if (p.info && wt == 0)
                    p.info[inst] = 0;
            }
            wg_barrier4(wg);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (tid < 32)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(cta.tmem_base), "r"(512) : "memory");
}

inline size_t smem4_bytes() { return SMEM4_BYTES; }

} // namespace umma64
} // namespace ttc
