// Riccati-backward + rollout kernel for n = m = 16 or 32, fp32 FFMA throughout.
//
// N lanes of a warp own one instance (two instances per warp when N = 16); lane c holds COLUMN c of
// every per-instance matrix in registers.  Because P, S, Q and R are symmetric, column c of them is
// also row c, so no transposition is ever needed:
//   V[:,c] = P B[:,c], T[:,c] = P A[:,c]      rows of P broadcast from the instance's scratch
//   S[:,c] = R[:,c] + B' V[:,c]               rows of B broadcast from the per-head operands
//   Y[:,c] = B' T[:,c],  Pn[:,c] = Q[:,c] + A' T[:,c]
//   S = L L'                                  warp-level Cholesky, one row per lane (row c = column c)
//   Z[:,c] = L^{-1} Y[:,c]                    in-lane forward substitution, columns of L broadcast
//   Pn[:,c] -= Z' Z[:,c]                      rows of Z broadcast          (P_t = Q + A'P A - Y'S^{-1}Y)
//   K[:,c] = -L^{-T} Z[:,c]                   in-lane back substitution (only when gains are needed)
// (Prop. 3.1; Alg. 1 backward loop), then the forward loop of Alg. 1 with one output row per lane.
// All cross-lane traffic goes through broadcast reads of shared memory rows (row stride N + 4 floats:
// 16-byte vector accesses by row owners and 4-byte accesses by column owners are both conflict-free).
//
// CTAs of 4 warps take chunks of consecutive tokens of one (sequence, head) from an atomic counter
// and keep that head's A, B, R in shared memory.
#pragma once

#include "common.cuh"

namespace ttc {
namespace rwarp {

constexpr int WARPS = 4;
constexpr int THREADS = 32 * WARPS;

template <int N>
struct Shape {
    static constexpr int LD = N + 4;               // row stride in floats
    static constexpr int IPW = 32 / N;             // instances per warp
    static constexpr int SLOTS = WARPS * IPW;      // instances in flight per CTA = tokens per chunk
    static constexpr int MAT = N * LD;
};

template <int N>
struct Smem {
    float A[Shape<N>::MAT], B[Shape<N>::MAT], R[Shape<N>::MAT];
    struct Slot {
        float buf0[Shape<N>::MAT];     // rows of P, then rows of Z
        float L[Shape<N>::MAT];        // rows of L
        float Lt[Shape<N>::MAT];       // rows of L' (columns of L); K_0 rows when only u_0 is wanted
        float rinv[N];                 // 1 / L[i][i]
        float x[N], u[N];
        float pv[N], gv[N];            // affine recursion (Prop. A.1): p_{t+1}, B'p_{t+1} + r_t
    } slot[Shape<N>::SLOTS];
    int chunk;
};

// Cholesky of an N x N SPD matrix spread over N lanes (lane i = row i = column i).  On return s holds
// row `c` of L (entries right of the diagonal are meaningless), rs_own = 1 / L[c][c].  The trailing
// update uses s_ij s_cj / d_j so that the broadcast of column j does not wait for the reciprocal.
// Returns 0 or 1 + the index of the first non-positive pivot.
template <int N>
__device__ __forceinline__ int seg_chol(float (&s)[N], float& rs_own, int c)
{
    int bad = 0;
    rs_own = 1.f;
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const float sj = s[j];
        float d = __shfl_sync(0xffffffffu, sj, j, N);
        if (!(d > 0.f)) {
            if (!bad)
                bad = j + 1;
            d = 1.f;
        }
        const float rinv = __frcp_rn(d);
        const float f = sj * rinv;
#pragma unroll
        for (int cc = j + 1; cc < N; ++cc) {
            const float lc = __shfl_sync(0xffffffffu, sj, cc, N);
            s[cc] = fmaf(-f, lc, s[cc]);
        }
        const float rs = rsqrtf(d);
        s[j] = sj * rs;
        if (c == j)
            rs_own = rs;
    }
    return bad;
}

template <int N>
__device__ __forceinline__ void load_row(float (&v)[N], const float* row)
{
#pragma unroll
    for (int q = 0; q < N / 4; ++q) {
        const float4 t = *reinterpret_cast<const float4*>(row + 4 * q);
        v[4 * q] = t.x; v[4 * q + 1] = t.y; v[4 * q + 2] = t.z; v[4 * q + 3] = t.w;
    }
}
template <int N>
__device__ __forceinline__ void store_row(float* row, const float (&v)[N])
{
#pragma unroll
    for (int q = 0; q < N / 4; ++q)
        *reinterpret_cast<float4*>(row + 4 * q) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
}
// row c of the (symmetric) Q of one instance, fp32 or bf16 in global memory
template <int N>
__device__ __forceinline__ void load_q_row(float (&q)[N], const OperandDev& Q, long long off)
{
    if (Q.dtype == TTC_BF16) {
        const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(Q.ptr) + off);
#pragma unroll
        for (int g = 0; g < N / 8; ++g) {
            const uint4 v = __ldg(src + g);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                q[8 * g + 2 * e] = __uint_as_float(w[e] << 16);
                q[8 * g + 2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
            }
        }
    } else {
        const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(Q.ptr) + off);
#pragma unroll
        for (int g = 0; g < N / 4; ++g) {
            const float4 v = __ldg(src + g);
            q[4 * g] = v.x; q[4 * g + 1] = v.y; q[4 * g + 2] = v.z; q[4 * g + 3] = v.w;
        }
    }
}
// ---- packed fp32 pairs: fma.rn.f32x2 does two FMAs per issued instruction (the dense loops are issue-bound)
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float a, float b)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& a, float& b)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ void fma2(f32x2& acc, f32x2 a, f32x2 b)
{
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}
template <int N>
__device__ __forceinline__ void pack_row(f32x2 (&v2)[N / 2], const float (&v)[N])
{
#pragma unroll
    for (int i = 0; i < N / 2; ++i)
        v2[i] = pack2(v[2 * i], v[2 * i + 1]);
}
template <int N>
__device__ __forceinline__ void unpack_row(float (&v)[N], const f32x2 (&v2)[N / 2])
{
#pragma unroll
    for (int i = 0; i < N / 2; ++i)
        unpack2(v2[i], v[2 * i], v[2 * i + 1]);
}
// acc[l] += w * row[l], l = 0..N-1
template <int N>
__device__ __forceinline__ void axpy_row(f32x2 (&acc)[N / 2], float w, const float* row)
{
    const f32x2 ww = pack2(w, w);
#pragma unroll
    for (int q = 0; q < N / 4; ++q) {
        const ulonglong2 t = *reinterpret_cast<const ulonglong2*>(row + 4 * q);
        fma2(acc[2 * q], ww, t.x);
        fma2(acc[2 * q + 1], ww, t.y);
    }
}

// ---- 32 x 32 x 32 contractions on the tensor cores (n = 32): mma.sync m16n8k8, tf32 operands, fp32 accumulate, with the
// operands split into tf32 high and low parts and three passes (lo*hi + hi*lo + hi*hi), which keeps float32-grade
// accuracy (the 1e-4 tolerance of the float32 configurations rules out single-pass tf32).  One warp computes one
// product; operands are float32 matrices in shared memory with row stride LD32 = 36 floats.
//   acc[mt][nt][..] is the 16 x 8 tile (rows 16 mt.., columns 8 nt..) in the accumulator layout of the instruction:
//   lane = 4 g + t holds (g, 2t), (g, 2t + 1), (g + 8, 2t), (g + 8, 2t + 1).
__device__ __forceinline__ void mma_tf32(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void split_hi_lo(float x, uint32_t& hi, uint32_t& lo)
{
    hi = __float_as_uint(x) & 0xffffe000u;
    lo = __float_as_uint(x - __uint_as_float(hi));
}
constexpr int LD32 = 36;
// acc += A' * B with both operands stored k-major: A'[i][k] = Am[k * LD32 + i], B[k][j] = Bm[k * LD32 + j].
// The instruction leaves the assignment of contraction indices to its k slots free as long as A and B agree, so
// slot (t, half) of k-step ks takes k = 16 (ks / 2) + 8 half + 2 t + (ks % 2): with the row stride of 36 floats the
// 32 lanes of a fragment load then fall into 32 different banks (bank = 8 t + g + 4 (ks % 2)).
__device__ __forceinline__ void mma32_product(float (&acc)[2][4][4], const float* Am, const float* Bm, int lane)
{
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
        const int k0 = 16 * (ks >> 1) + 2 * t + (ks & 1);
        uint32_t ah[2][4], al[2][4], bh[4][2], bl[4][2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const int i0 = 16 * mt + g;
            split_hi_lo(Am[k0 * LD32 + i0], ah[mt][0], al[mt][0]);
            split_hi_lo(Am[k0 * LD32 + i0 + 8], ah[mt][1], al[mt][1]);
            split_hi_lo(Am[(k0 + 8) * LD32 + i0], ah[mt][2], al[mt][2]);
            split_hi_lo(Am[(k0 + 8) * LD32 + i0 + 8], ah[mt][3], al[mt][3]);
        }
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            split_hi_lo(Bm[k0 * LD32 + 8 * nt + g], bh[nt][0], bl[nt][0]);
            split_hi_lo(Bm[(k0 + 8) * LD32 + 8 * nt + g], bh[nt][1], bl[nt][1]);
        }
        // pass-major order: the eight accumulator tiles of a pass are independent of one another
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
                mma_tf32(acc[mt][nt], al[mt][0], al[mt][1], al[mt][2], al[mt][3], bh[nt][0], bh[nt][1]);
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
                mma_tf32(acc[mt][nt], ah[mt][0], ah[mt][1], ah[mt][2], ah[mt][3], bl[nt][0], bl[nt][1]);
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
                mma_tf32(acc[mt][nt], ah[mt][0], ah[mt][1], ah[mt][2], ah[mt][3], bh[nt][0], bh[nt][1]);
    }
}
__device__ __forceinline__ void mma32_zero(float (&acc)[2][4][4])
{
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                acc[mt][nt][e] = 0.f;
}
// accumulator tiles -> row-major matrix in shared memory (8-byte stores)
__device__ __forceinline__ void mma32_store(float* Dm, const float (&acc)[2][4][4], int lane)
{
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            *reinterpret_cast<float2*>(Dm + (16 * mt + g) * LD32 + 8 * nt + 2 * t) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
            *reinterpret_cast<float2*>(Dm + (16 * mt + g + 8) * LD32 + 8 * nt + 2 * t) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
        }
}

// Per-head operands of time index t -> shared memory (all threads of the CTA; the caller synchronises).
template <int N>
__device__ __forceinline__ void load_head_operands(Smem<N>& sm, const SolveParams& p, long long oa, long long ob, long long orr,
                                                   int t, bool la, bool lb, bool lr)
{
    constexpr int LD = Shape<N>::LD;
    const float* Ag = reinterpret_cast<const float*>(p.A.ptr) + oa + t * p.A.st;
    const float* Bg = reinterpret_cast<const float*>(p.B.ptr) + ob + t * p.B.st;
    const float* Rg = reinterpret_cast<const float*>(p.R.ptr) + orr + t * p.R.st;
    for (int e = threadIdx.x; e < N * N; e += THREADS) {
        const int r = e / N, cc = e % N;
        if (la) sm.A[r * LD + cc] = __ldg(Ag + e);
        if (lb) sm.B[r * LD + cc] = __ldg(Bg + e);
        if (lr) sm.R[r * LD + cc] = __ldg(Rg + e);
    }
}

// Operands of ONE instance at time index t -> that instance's own copies (its N lanes; the caller synchronises the
// segment).  Lane c takes column c of every row: N consecutive floats per request.
template <int N>
__device__ __forceinline__ void load_slot_operands(float* As, float* Bs, float* Rs, const SolveParams& p, long long oa,
                                                   long long ob, long long orr, int t, bool la, bool lb, bool lr, int c)
{
    constexpr int LD = Shape<N>::LD;
    const float* Ag = reinterpret_cast<const float*>(p.A.ptr) + oa + t * p.A.st;
    const float* Bg = reinterpret_cast<const float*>(p.B.ptr) + ob + t * p.B.st;
    const float* Rg = reinterpret_cast<const float*>(p.R.ptr) + orr + t * p.R.st;
#pragma unroll 4
    for (int k = 0; k < N; ++k) {
        if (la) As[k * LD + c] = __ldg(Ag + k * N + c);
        if (lb) Bs[k * LD + c] = __ldg(Bg + k * N + c);
        if (lr) Rs[k * LD + c] = __ldg(Rg + k * N + c);
    }
}

// TV = time-varying request (time strides or a terminal weight): the other instantiation carries none of that code.
// AFF = linear control cost r_t'u_t (Prop. A.1: p_t, k_t); implies TV.
// PT = A, B, R belong to the token, not to the head (the contextualised layer's situation): every instance keeps its own
// copies behind the common part of shared memory and its lanes reload them; implies TV.
template <int N, bool TV, bool AFF = false, bool PT = false>
__global__ void __launch_bounds__(THREADS, (N == 32) ? 3 : 4) riccati_warp_kernel(SolveParams p, int* chunk_counter)
{
    using S = Shape<N>;
    constexpr int LD = S::LD;
    // n = 32: the dense contractions of a step run on the tensor cores (mma.sync, three-pass tf32); the factorisation,
    // the substitutions, the vector recursion of the affine term and the rollout stay on the FP32 pipe
    constexpr bool MMA = (N == 32);
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem<N>& sm = *reinterpret_cast<Smem<N>*>(smem_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sub = lane / N, c = lane % N;
    typename Smem<N>::Slot& sl = sm.slot[warp * S::IPW + sub];
    float* own_ops = reinterpret_cast<float*>(smem_raw + ((sizeof(Smem<N>) + 15) & ~size_t(15))) + (warp * S::IPW + sub) * 3 * S::MAT;
    float* const As = PT ? own_ops : sm.A;
    float* const Bs = PT ? own_ops + S::MAT : sm.B;
    float* const Rs = PT ? own_ops + 2 * S::MAT : sm.R;
    const int H = p.H;
    const long long chunks_per_head = (p.tcount + S::SLOTS - 1) / S::SLOTS;
    const long long nchunks = p.b0 * p.b1 * chunks_per_head;
    const bool need_K_all = (p.K != nullptr) || (p.x != nullptr) || (p.u != nullptr && !p.first_only);
    const bool want_u0 = (p.u != nullptr) && p.first_only && !need_K_all;
    const bool need_k_all = AFF && p.kff != nullptr;          // feed-forward terms wanted (output or rollout)
    // With bfloat16 outputs the rollout still reads float32 gains: they go to the workspace, and to K as bfloat16 too.
    const int obf = p.out_bf16;
    float* Kbase = (p.K && !obf) ? p.K : p.Kws;
    long long offA = -1, offB = -1, offR = -1;

    for (;;) {
        __syncthreads();
        if (tid == 0)
            sm.chunk = atomicAdd(chunk_counter, 1);
        __syncthreads();
        const long long chunk = sm.chunk;
        if (chunk >= nchunks)
            break;
        const long long head = chunk / chunks_per_head;
        const long long tok0 = p.t0 + (chunk % chunks_per_head) * S::SLOTS;
        const long long inst0 = head * p.b2 + tok0;
        const int ntok = (int)min((long long)S::SLOTS, p.t0 + p.tcount - tok0);
        const long long oa = operand_offset(p.A, inst0, p.b1, p.b2);
        const long long ob = operand_offset(p.B, inst0, p.b1, p.b2);
        const long long orr = operand_offset(p.R, inst0, p.b1, p.b2);
        const bool tv_head = TV && (p.A.st | p.B.st | p.R.st) != 0;      // the operands change with the time index
        if (!PT && (tv_head || oa != offA || ob != offB || orr != offR)) {
            load_head_operands<N>(sm, p, oa, ob, orr, TV ? H - 1 : 0, true, true, true);
            offA = oa; offB = ob; offR = orr;
        }
        __syncthreads();
        const int slot_idx = warp * S::IPW + sub;
        const bool active = slot_idx < ntok;                  // idle segments shadow the chunk's first instance
        const long long inst = inst0 + (active ? slot_idx : 0);
        const long long oai = PT ? operand_offset(p.A, inst, p.b1, p.b2) : oa;
        const long long obi = PT ? operand_offset(p.B, inst, p.b1, p.b2) : ob;
        const long long ori = PT ? operand_offset(p.R, inst, p.b1, p.b2) : orr;
        if (PT)
            load_slot_operands<N>(As, Bs, Rs, p, oai, obi, ori, H - 1, true, true, true, c);    // ordered by the barrier below
        const long long oq = operand_offset(p.Q, inst, p.b1, p.b2) + (long long)c * N;

        const bool wantP = p.P && active;
        const long long Poff = inst * (long long)(p.first_only ? 1 : H + 1) * N * N;     // first element of this instance's P
        float* Kout = (Kbase && need_K_all) ? Kbase + inst * (long long)H * N * N : nullptr;
        float pcol[N];
        if (TV && p.Qf.ptr)
            load_q_row<N>(pcol, p.Qf, operand_offset(p.Qf, inst, p.b1, p.b2) + (long long)c * N);   // P_H = Q_f
        else
            load_q_row<N>(pcol, p.Q, oq);                     // P_H = Q
        if (wantP && !p.first_only) {
#pragma unroll
            for (int l = 0; l < N; ++l)
                store_out(p.P, Poff + (long long)H * N * N + l * N + c, pcol[l], obf);
        }
        store_row<N>(sl.buf0 + c * LD, pcol);
        if (p.x0.ptr)
            sl.x[c] = load_elem(p.x0, operand_offset(p.x0, inst, p.b1, p.b2) + c);
        float k0c = 0.f;                                      // k_0[c] when only u_0 is wanted
        const long long orv = AFF ? operand_offset(p.r, inst, p.b1, p.b2) + c : 0;
        if (AFF) {
            sl.pv[c] = 0.f;                                   // p_H = 0
            if (p.pvec && !p.first_only && active)
                p.pvec[inst * (long long)(H + 1) * N + (long long)H * N + c] = 0.f;
        }
        __syncwarp();
        int fail = 0;

#pragma unroll 1
        for (int ts = H - 1; ts >= 0; --ts) {
            if (tv_head && ts != H - 1) {                     // A_t, B_t, R_t of this step
                if (PT) {
                    __syncwarp();
                    load_slot_operands<N>(As, Bs, Rs, p, oai, obi, ori, ts, p.A.st != 0, p.B.st != 0, p.R.st != 0, c);
                    __syncwarp();
                } else {                                      // the whole CTA is in step
                    __syncthreads();
                    load_head_operands<N>(sm, p, oa, ob, orr, ts, p.A.st != 0, p.B.st != 0, p.R.st != 0);
                    __syncthreads();
                }
            }
            float s[N], y[N];
            f32x2 p2[N / 2];
            float pn[N];                                      // tensor-core path: column c of Q_t + A'T
            // Tensor-core path: the six 32 x 32 x 32 products of a step (V = P B, T = P A, S - R = B'V, Y = B'T, A'T,
            // Z'Z) share one copy of the product code: phases 0..4 run it on the way to the factorisation, phase 5 first
            // factorises and substitutes, then runs it on Z.  Straight-line code for every product separately does not
            // fit the instruction cache next to the unrolled factorisation.  Without tensor cores there is only phase 5.
#pragma unroll 1
            for (int ph = MMA ? 0 : 5; ph < 6; ++ph) {
            if (!MMA || ph == 5) {
            if constexpr (MMA) {
                float tmp[N];
                load_row<N>(s, Rs + c * LD);                  // S[:,c] = R[:,c] + (B'V)[c,:]  (symmetric)
                load_row<N>(tmp, sl.buf0 + c * LD);
                load_q_row<N>(pn, p.Q, TV ? oq + ts * p.Q.st : oq);
#pragma unroll
                for (int l = 0; l < N; ++l) {
                    s[l] += tmp[l];
                    y[l] = sl.L[l * LD + c];
                    pn[l] += sl.Lt[l * LD + c];
                }
            } else {
                f32x2 vcol[N / 2], tcol[N / 2];
#pragma unroll
                for (int k = 0; k < N / 2; ++k) {
                    vcol[k] = 0ull;
                    tcol[k] = 0ull;
                }
#pragma unroll 4
                for (int i = 0; i < N; ++i) {                     // V[:,c] = P B[:,c], T[:,c] = P A[:,c]
                    const float bic = Bs[i * LD + c], aic = As[i * LD + c];
                    const f32x2 b2 = pack2(bic, bic), a2 = pack2(aic, aic);
                    const float* prow = sl.buf0 + i * LD;
#pragma unroll
                    for (int q = 0; q < N / 4; ++q) {
                        const ulonglong2 t = *reinterpret_cast<const ulonglong2*>(prow + 4 * q);
                        fma2(vcol[2 * q], t.x, b2);
                        fma2(vcol[2 * q + 1], t.y, b2);
                        fma2(tcol[2 * q], t.x, a2);
                        fma2(tcol[2 * q + 1], t.y, a2);
                    }
                }
                // stage the two columns in the instance's scratch (own column only: no exchange) so that the next loop
                // can run over k without indexing registers dynamically
#pragma unroll
                for (int k = 0; k < N / 2; ++k) {
                    float v0, v1, t0, t1;
                    unpack2(vcol[k], v0, v1);
                    unpack2(tcol[k], t0, t1);
                    sl.L[(2 * k) * LD + c] = v0;
                    sl.L[(2 * k + 1) * LD + c] = v1;
                    sl.Lt[(2 * k) * LD + c] = t0;
                    sl.Lt[(2 * k + 1) * LD + c] = t1;
                }
                f32x2 s2[N / 2], y2[N / 2];
                {
                    float tmp[N];
                    load_row<N>(tmp, Rs + c * LD);              // S[:,c] = R[:,c] + B' V[:,c]
                    pack_row<N>(s2, tmp);
                    load_q_row<N>(tmp, p.Q, TV ? oq + ts * p.Q.st : oq);    // Pn[:,c] = Q_t[:,c] + A' T[:,c] ; Y[:,c] = B' T[:,c]
                    pack_row<N>(p2, tmp);
                }
#pragma unroll
                for (int l = 0; l < N / 2; ++l)
                    y2[l] = 0ull;
#pragma unroll 4
                for (int k = 0; k < N; ++k) {
                    const float vk = sl.L[k * LD + c], tk = sl.Lt[k * LD + c];
                    const f32x2 vv = pack2(vk, vk), tt = pack2(tk, tk);
#pragma unroll
                    for (int q = 0; q < N / 4; ++q) {             // each row of B and A is read once
                        const ulonglong2 b4 = *reinterpret_cast<const ulonglong2*>(Bs + k * LD + 4 * q);
                        const ulonglong2 a4 = *reinterpret_cast<const ulonglong2*>(As + k * LD + 4 * q);
                        fma2(s2[2 * q], vv, b4.x);
                        fma2(s2[2 * q + 1], vv, b4.y);
                        fma2(y2[2 * q], tt, b4.x);
                        fma2(y2[2 * q + 1], tt, b4.y);
                        fma2(p2[2 * q], tt, a4.x);
                        fma2(p2[2 * q + 1], tt, a4.y);
                    }
                }
                unpack_row<N>(s, s2);
                unpack_row<N>(y, y2);
            }
            float gz[N];                                      // B'p + r, then L^{-1}(.), then k_t = -S^{-1}(.) (every lane holds all of it)
            float apc = 0.f;                                  // (A'p_{t+1})[c]
            if (AFF) {
                float pvv[N];
                load_row<N>(pvv, sl.pv);
                float gc = ts < p.r_count ? load_elem(p.r, orv + ts * p.r.st) : 0.f;
#pragma unroll
                for (int i = 0; i < N; ++i) {
                    gc = fmaf(Bs[i * LD + c], pvv[i], gc);
                    apc = fmaf(As[i * LD + c], pvv[i], apc);
                }
                sl.gv[c] = gc;
            }
            float rs_own;
            const int bad = seg_chol<N>(s, rs_own, c);
            if (bad && !fail)
                fail = ts * N + bad;
            __syncwarp();                                     // every lane is done with the rows of P in buf0
            store_row<N>(sl.L + c * LD, s);
#pragma unroll
            for (int k = 0; k < N; ++k)
                sl.Lt[k * LD + c] = s[k];
            sl.rinv[c] = rs_own;
            __syncwarp();
            float rinv[N];
            load_row<N>(rinv, sl.rinv);
            if (AFF)
                load_row<N>(gz, sl.gv);
#pragma unroll
            for (int k = 0; k < N; ++k) {                     // Z[:,c] = L^{-1} Y[:,c]  (and L^{-1}(B'p + r))
                const float zk = y[k] * rinv[k];
                y[k] = zk;
                float zg = 0.f;
                if (AFF) {
                    zg = gz[k] * rinv[k];
                    gz[k] = zg;
                }
                const float* lt = sl.Lt + k * LD;
#pragma unroll
                for (int i4 = (k + 1) & ~3; i4 < N; i4 += 4) {
                    const float4 l4 = *reinterpret_cast<const float4*>(lt + i4);
                    if (i4 + 0 > k) y[i4 + 0] = fmaf(-l4.x, zk, y[i4 + 0]);
                    if (i4 + 1 > k) y[i4 + 1] = fmaf(-l4.y, zk, y[i4 + 1]);
                    if (i4 + 2 > k) y[i4 + 2] = fmaf(-l4.z, zk, y[i4 + 2]);
                    if (i4 + 3 > k) y[i4 + 3] = fmaf(-l4.w, zk, y[i4 + 3]);
                    if (AFF) {
                        if (i4 + 0 > k) gz[i4 + 0] = fmaf(-l4.x, zg, gz[i4 + 0]);
                        if (i4 + 1 > k) gz[i4 + 1] = fmaf(-l4.y, zg, gz[i4 + 1]);
                        if (i4 + 2 > k) gz[i4 + 2] = fmaf(-l4.z, zg, gz[i4 + 2]);
                        if (i4 + 3 > k) gz[i4 + 3] = fmaf(-l4.w, zg, gz[i4 + 3]);
                    }
                }
            }
            if (AFF) {                                        // p_t[c] = (A'p_{t+1})[c] - Z[:,c] . L^{-1}(B'p_{t+1} + r_t)
                float pc = apc;
#pragma unroll
                for (int q = 0; q < N; ++q)
                    pc = fmaf(-y[q], gz[q], pc);
                sl.pv[c] = pc;                                // every lane has read p_{t+1} before the barriers above
                if (p.pvec && active && (!p.first_only || ts == 0))
                    p.pvec[inst * (long long)(p.first_only ? 1 : H + 1) * N + (long long)(p.first_only ? 0 : ts) * N + c] = pc;
            }
#pragma unroll
            for (int q = 0; q < N; ++q)
                sl.buf0[q * LD + c] = y[q];                   // rows of Z
            __syncwarp();
            if constexpr (!MMA) {
#pragma unroll 4
                for (int q = 0; q < N; ++q)                   // Pn[:,c] -= Z' Z[:,c]
                    axpy_row<N>(p2, -sl.buf0[q * LD + c], sl.buf0 + q * LD);
                unpack_row<N>(pcol, p2);
            }
            const bool gains = need_K_all || need_k_all || (want_u0 && ts == 0);
            if (gains) {                                      // K[:,c] = -L^{-T} Z[:,c]  (and k_t = -L^{-T} L^{-1}(B'p + r))
#pragma unroll
                for (int k = N - 1; k >= 0; --k) {
                    const float xk = y[k] * rinv[k];
                    y[k] = xk;
                    float xg = 0.f;
                    if (AFF) {
                        xg = gz[k] * rinv[k];
                        gz[k] = xg;
                    }
                    const float* lr = sl.L + k * LD;
#pragma unroll
                    for (int i4 = 0; i4 < k; i4 += 4) {
                        const float4 l4 = *reinterpret_cast<const float4*>(lr + i4);
                        if (i4 + 0 < k) y[i4 + 0] = fmaf(-l4.x, xk, y[i4 + 0]);
                        if (i4 + 1 < k) y[i4 + 1] = fmaf(-l4.y, xk, y[i4 + 1]);
                        if (i4 + 2 < k) y[i4 + 2] = fmaf(-l4.z, xk, y[i4 + 2]);
                        if (i4 + 3 < k) y[i4 + 3] = fmaf(-l4.w, xk, y[i4 + 3]);
                        if (AFF) {
                            if (i4 + 0 < k) gz[i4 + 0] = fmaf(-l4.x, xg, gz[i4 + 0]);
                            if (i4 + 1 < k) gz[i4 + 1] = fmaf(-l4.y, xg, gz[i4 + 1]);
                            if (i4 + 2 < k) gz[i4 + 2] = fmaf(-l4.z, xg, gz[i4 + 2]);
                            if (i4 + 3 < k) gz[i4 + 3] = fmaf(-l4.w, xg, gz[i4 + 3]);
                        }
                    }
                }
                if (AFF) {
                    float kc = 0.f;
#pragma unroll
                    for (int l = 0; l < N; ++l)
                        if (l == c)
                            kc = -gz[l];
                    if (ts == 0)
                        k0c = kc;
                    if (need_k_all && active)
                        p.kff[(inst * (long long)H + ts) * N + c] = kc;
                }
                if (need_K_all) {
                    if (active) {
                        float* kt = Kout + (long long)ts * N * N + c;
#pragma unroll
                        for (int l = 0; l < N; ++l)
                            kt[l * N] = -y[l];
                        if (obf && p.K) {
                            const long long ko = (inst * (long long)H + ts) * N * N + c;
#pragma unroll
                            for (int l = 0; l < N; ++l)
                                store_out(p.K, ko + l * N, -y[l], 1);
                        }
                    }
                } else if (want_u0 && ts == 0) {              // K_0 rows -> Lt (free after the forward substitution)
#pragma unroll
                    for (int l = 0; l < N; ++l)
                        sl.Lt[l * LD + c] = -y[l];
                }
            }
            }                                                 // phase 5: factorisation, substitutions, gains
            if constexpr (MMA) {
                // phase:  0      1      2      3      4      5
                // A'   :  P      P      B'     B'     A'     Z'          (P symmetric, so P B = P'B)
                // B    :  B      A      V      T      T      Z
                // to   :  L      L'     buf0   L      L'     L           (buf0: P, then B'V, then Z)
                // The rows of L' may hold K_0 for the last step's u_0, so Z'Z goes to the rows of L.
                const float* Am = ph < 2 ? sl.buf0 : ph == 4 ? As : ph == 5 ? sl.buf0 : Bs;
                const float* Bm = ph == 0 ? Bs : ph == 1 ? As : ph == 2 ? sl.L : ph == 5 ? sl.buf0 : sl.Lt;
                float* Dm = ph == 1 || ph == 4 ? sl.Lt : ph == 2 ? sl.buf0 : sl.L;
                float acc[2][4][4];
                mma32_zero(acc);
                mma32_product(acc, Am, Bm, lane);
                __syncwarp();                                 // every lane has read what the result overwrites
                mma32_store(Dm, acc, lane);
                __syncwarp();
                if (ph == 5) {
#pragma unroll
                    for (int l = 0; l < N; ++l)
                        pcol[l] = pn[l] - sl.L[l * LD + c];   // P_t[:,c] = Q[:,c] + A'T[:,c] - Z'Z[:,c]
                }
            }
            }                                                 // phases
            __syncwarp();                                     // rows of Z consumed
            store_row<N>(sl.buf0 + c * LD, pcol);             // column c of P_t as row c
            __syncwarp();
            // P_t <- (P_t + P_t') / 2.  Q_t and Z'Z are symmetric, but the rounding of A'(P A) is not, and since the next
            // step reads the rows above as columns, the antisymmetric part E obeys E <- -A'E A: it grows along an
            // open-loop unstable A (|eig| > 1) however well the closed loop is damped, and takes over long horizons.
#pragma unroll
            for (int l = 0; l < N; ++l)
                pcol[l] = 0.5f * (pcol[l] + sl.buf0[l * LD + c]);
            if (wantP && (!p.first_only || ts == 0)) {
                const long long po = Poff + (long long)(p.first_only ? 0 : ts) * N * N + c;
#pragma unroll
                for (int l = 0; l < N; ++l)
                    store_out(p.P, po + l * N, pcol[l], obf);
            }
            __syncwarp();                                     // every lane has read its column
            store_row<N>(sl.buf0 + c * LD, pcol);
            __syncwarp();
        }

        // A failure is known to every lane of the segment.  Control flow stays warp-uniform (the two
        // segments of a warp may differ): a failed instance only loses its stores.
        if (fail && active) {
            const float qn = quiet_nan();
            if (p.K)
                for (long long e = c; e < (long long)H * N * N; e += N)
                    store_out(p.K, inst * (long long)H * N * N + e, qn, obf);
            if (p.P) {
                const long long cnt = (long long)(p.first_only ? 1 : H + 1) * N * N;
                for (long long e = c; e < cnt; e += N)
                    store_out(p.P, inst * cnt + e, qn, obf);
            }
            if (p.x)
                for (long long e = c; e < (long long)(H + 1) * N; e += N)
                    store_out(p.x, inst * (long long)(H + 1) * N + e, qn, obf);
            if (p.u) {
                const long long cnt = p.first_only ? N : (long long)H * N;
                for (long long e = c; e < cnt; e += N)
                    store_out(p.u, inst * cnt + e, qn, obf);
            }
            if (AFF && p.pvec) {
                const long long cnt = (long long)(p.first_only ? 1 : H + 1) * N;
                for (long long e = c; e < cnt; e += N)
                    p.pvec[inst * cnt + e] = qn;
            }
            if (need_k_all)
                for (long long e = c; e < (long long)H * N; e += N)
                    p.kff[inst * (long long)H * N + e] = qn;
        }
        if (p.info && active && c == 0)
            p.info[inst] = fail;
        const bool store_ok = active && !fail;

        // ---- forward loop of Alg. 1: lane c computes u_t[c] and x_{t+1}[c]
        if (want_u0) {
            float kr[N], xv[N];
            load_row<N>(kr, sl.Lt + c * LD);
            load_row<N>(xv, sl.x);
            float uc = AFF ? k0c : 0.f;                       // u_0 = K_0 x_0 + k_0
#pragma unroll
            for (int j = 0; j < N; ++j)
                uc = fmaf(kr[j], xv[j], uc);
            if (store_ok)
                store_out(p.u, inst * (long long)N + c, uc, obf);
        } else if (p.x || p.u) {
            const bool xo = p.x && store_ok, uo = p.u && store_ok;
            const long long xoff = inst * (long long)(H + 1) * N, uoff = inst * (long long)(p.first_only ? N : H * N);
            float arow[N], brow[N];
            if (!tv_head) {
                load_row<N>(arow, As + c * LD);
                load_row<N>(brow, Bs + c * LD);
            }
            if (xo)
                store_out(p.x, xoff + c, sl.x[c], obf);
            __syncwarp();                                     // K_t written by the other lanes are visible
#pragma unroll 1
            for (int ts = 0; ts < H; ++ts) {
                if (tv_head) {                                // A_t, B_t of this step (after the backward pass they hold t = 0)
                    if (ts > 0) {
                        if (PT) {
                            __syncwarp();
                            load_slot_operands<N>(As, Bs, Rs, p, oai, obi, ori, ts, p.A.st != 0, p.B.st != 0, false, c);
                            __syncwarp();
                        } else {
                            __syncthreads();
                            load_head_operands<N>(sm, p, oa, ob, orr, ts, p.A.st != 0, p.B.st != 0, false);
                            __syncthreads();
                        }
                    }
                    load_row<N>(arow, As + c * LD);
                    load_row<N>(brow, Bs + c * LD);
                }
                float xv[N];
                load_row<N>(xv, sl.x);
                const float4* kr = reinterpret_cast<const float4*>(Kout + (long long)ts * N * N + c * N);
                float uc = need_k_all ? p.kff[(inst * (long long)H + ts) * N + c]        // own store of the backward pass
                                      : (AFF && ts == 0) ? k0c : 0.f;
#pragma unroll
                for (int q = 0; q < N / 4; ++q) {
                    const float4 k4 = kr[q];
                    uc = fmaf(k4.x, xv[4 * q], uc);
                    uc = fmaf(k4.y, xv[4 * q + 1], uc);
                    uc = fmaf(k4.z, xv[4 * q + 2], uc);
                    uc = fmaf(k4.w, xv[4 * q + 3], uc);
                }
                sl.u[c] = uc;
                if (uo && (!p.first_only || ts == 0))
                    store_out(p.u, uoff + (p.first_only ? 0 : ts * N) + c, uc, obf);
                __syncwarp();
                float uv[N];
                load_row<N>(uv, sl.u);
                float xc = 0.f;
#pragma unroll
                for (int j = 0; j < N; ++j)
                    xc = fmaf(arow[j], xv[j], fmaf(brow[j], uv[j], xc));
                __syncwarp();                                 // x_t consumed by every lane
                sl.x[c] = xc;
                if (xo)
                    store_out(p.x, xoff + (long long)(ts + 1) * N + c, xc, obf);
                __syncwarp();
            }
        }
    }
}

template <int N>
inline size_t smem_bytes(bool per_token = false)
{
    // the per-token copies start on the next 16-byte boundary: their rows are read with 16-byte loads
    return per_token ? ((sizeof(Smem<N>) + 15) & ~size_t(15)) + sizeof(float) * Shape<N>::SLOTS * 3 * Shape<N>::MAT : sizeof(Smem<N>);
}

} // namespace rwarp
} // namespace ttc
