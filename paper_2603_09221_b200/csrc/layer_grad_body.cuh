// Body of layer_grad_vectors_kernel (included by layer_grad.cuh): rollouts forward, co-states and reductions backward.
#pragma once

namespace ttc {
namespace lgrad {

template <int N>
__global__ void __launch_bounds__(THREADS, (N == 32) ? 2 : 4) layer_grad_vectors_kernel(LayerGradParams q)
{
    using S = Shape<N>;
    constexpr int LD = S::LD;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const layer::LayerParams& p = q.lp;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, sub = lane / N, c = lane % N;
    Slot<N>& sl = reinterpret_cast<Slot<N>*>(smem_raw)[warp * S::IPW + sub];
    const int T = p.T, r = p.r;
    for (long long base = (long long)blockIdx.x * S::SLOTS; base < p.N; base += (long long)gridDim.x * S::SLOTS) {
        const long long raw = base + warp * S::IPW + sub;
        const bool active = raw < p.N;
        const long long inst = active ? raw : base;
        const bool failed = q.info[inst] != 0;
        __syncwarp();
        // ---- synthesis: column c of Bbar (kept in registers too), rows of Bbar, Qbar, Q_T in the slot
        float bcol[N];
        {
            float qcol[N], fcol[N];
#pragma unroll
            for (int l = 0; l < N; ++l) {
                bcol[l] = 0.f;
                qcol[l] = 0.f;
                fcol[l] = 0.f;
            }
#pragma unroll 1
            for (int i = 0; i < r; ++i) {
                const float wb = __ldg(p.s_b + inst * r + i), wq = __ldg(p.s_q + inst * r + i), wf = __ldg(p.s_qf + inst * r + i);
                const float* Bi = p.B_basis + (long long)i * N * N + c;
                const float* Qi = p.Q_basis + (long long)i * N * N + c;
#pragma unroll
                for (int l = 0; l < N; ++l) {
                    const float qv = __ldg(Qi + l * N);
                    bcol[l] = fmaf(wb, __ldg(Bi + l * N), bcol[l]);
                    qcol[l] = fmaf(wq, qv, qcol[l]);
                    fcol[l] = fmaf(wf, qv, fcol[l]);
                }
            }
#pragma unroll
            for (int l = 0; l < N; ++l) {
                sl.Bb[l * LD + c] = bcol[l];
                sl.Qb[l * LD + c] = qcol[l];
                sl.Qf[l * LD + c] = fcol[l];
            }
        }
        const float sa_c = __ldg(p.s_a + inst * N + c), ga_c = __ldg(p.s_ga + inst * N + c);
        const float gb_c = __ldg(p.s_gb + inst * N + c), gq_c = __ldg(p.s_gq + inst * N + c);
        const float ri_c = __ldg(p.r_inv + inst * N + c);
        float* X = q.vec + inst * (long long)(4 * (T + 1)) * N;       // x_s | xd_s | u_s | ud_s, (T + 1) rows of N each
        float* Xd = X + (long long)(T + 1) * N;
        float* U = Xd + (long long)(T + 1) * N;
        float* Ud = U + (long long)(T + 1) * N;
        // ---- forward: primal rollout from h_0, dual rollout from 0 with the first control k_0 (Prop. A.1, r_0 = g)
        {
            const float h = __ldg(p.h0 + inst * N + c);
            sl.x[c] = h;
            sl.xd[c] = 0.f;
            if (active) {
                X[c] = h;
                Xd[c] = 0.f;
            }
        }
        __syncwarp();
#pragma unroll 1
        for (int s = 0; s < T; ++s) {
            float xv[N], xdv[N], krow[N];
            load_row<N>(xv, sl.x);
            load_row<N>(xdv, sl.xd);
            load_vec_global<N>(krow, p.Kws + (inst * (long long)T + s) * N * N + c * N);
            float uc = 0.f, udc = (s == 0) ? __ldg(p.k0 + inst * N + c) : 0.f;
#pragma unroll
            for (int j = 0; j < N; ++j) {
                uc = fmaf(krow[j], xv[j], uc);
                udc = fmaf(krow[j], xdv[j], udc);
            }
            const float tt = (float)(s + 1);
            const float g_c = __expf(-tt * gb_c);
            const float a_c = fmaf(__expf(-tt * ga_c), sa_c, 1.f);
            sl.gu[c] = g_c * uc;
            sl.gud[c] = g_c * udc;
            if (active) {
                U[(long long)s * N + c] = uc;
                Ud[(long long)s * N + c] = udc;
            }
            __syncwarp();
            float gv[N], gdv[N];
            load_row<N>(gv, sl.gu);
            load_row<N>(gdv, sl.gud);
            const float xn = fmaf(a_c, sl.x[c], dot_row<N>(sl.Bb + c * LD, gv));       // a_s x_s[c] + (Bbar (g .* u))[c]
            const float xdn = fmaf(a_c, sl.xd[c], dot_row<N>(sl.Bb + c * LD, gdv));
            __syncwarp();                                     // x_s, xd_s consumed by every lane
            sl.x[c] = xn;
            sl.xd[c] = xdn;
            if (active) {
                X[(long long)(s + 1) * N + c] = xn;
                Xd[(long long)(s + 1) * N + c] = xdn;
            }
            __syncwarp();
        }
        // ---- backward: co-states of both problems, every outer product of Thm 3.2 reduced as it appears
        float dB[N], dQ[N], dF[N];                            // column c of the gradients of Bbar, Qbar, Q_T
        float d_sa = 0.f, d_ga = 0.f, d_gb = 0.f, d_gq = 0.f, d_ri = 0.f;
        float lam_c, lamd_c;
        {
            float xv[N], xdv[N];
            load_row<N>(xv, sl.x);                            // x_T, xd_T
            load_row<N>(xdv, sl.xd);
            lam_c = dot_row<N>(sl.Qf + c * LD, xv);           // lam_T = Q_T x_T (row c of the symmetric Q_T)
            lamd_c = dot_row<N>(sl.Qf + c * LD, xdv);
            const float xc = sl.x[c], xdc = sl.xd[c];
#pragma unroll
            for (int i = 0; i < N; ++i) {
                dF[i] = 0.5f * (xv[i] * xdc + xdv[i] * xc);
                dB[i] = 0.f;
                dQ[i] = 0.f;
            }
        }
        __syncwarp();
        sl.lam[c] = lam_c;
        sl.lamd[c] = lamd_c;
        __syncwarp();
#pragma unroll 1
        for (int s = T - 1; s >= 0; --s) {
            const float tt = (float)(s + 1), ts = (float)s;
            const float ea = __expf(-tt * ga_c), g_c = __expf(-tt * gb_c);
            const float a_c = fmaf(ea, sa_c, 1.f);
            if (s + 1 < T) {
                // co-states as lam_{s+1} = P_{s+1} x_{s+1} (and the same for the dual, whose linear term vanishes from
                // s = 1 on): the recursion lam_s = a_s lam_{s+1} + Q_s x_s would amplify rounding by the open-loop a_s
                float pr[N], xn[N], xdn[N];
                load_vec_global<N>(pr, p.Pws + (inst * (long long)T + s + 1) * N * N + c * N);
                load_vec_plain<N>(xn, X + (long long)(s + 1) * N);
                load_vec_plain<N>(xdn, Xd + (long long)(s + 1) * N);
                lam_c = 0.f;
                lamd_c = 0.f;
#pragma unroll
                for (int j = 0; j < N; ++j) {
                    lam_c = fmaf(pr[j], xn[j], lam_c);
                    lamd_c = fmaf(pr[j], xdn[j], lamd_c);
                }
                __syncwarp();                                 // the previous step's reads of the co-state vectors are done
                sl.lam[c] = lam_c;
                sl.lamd[c] = lamd_c;
                __syncwarp();
            }
            float xv[N], xdv[N];
            load_vec_plain<N>(xv, X + (long long)s * N);       // written by this kernel: ordinary loads
            load_vec_plain<N>(xdv, Xd + (long long)s * N);
            const float uc = U[(long long)s * N + c], udc = Ud[(long long)s * N + c];
            float xc = 0.f, xdc = 0.f;
#pragma unroll
            for (int i = 0; i < N; ++i)
                if (i == c) {
                    xc = xv[i];
                    xdc = xdv[i];
                }
            const float dA = fmaf(lam_c, xdc, lamd_c * xc);   // dA_s[c][c]
            d_sa = fmaf(ea, dA, d_sa);
            d_ga = fmaf(-tt * ea * sa_c, dA, d_ga);
            d_ri = fmaf(-uc, udc, d_ri);
            {
                float lv[N], ldv[N];
                load_row<N>(lv, sl.lam);
                load_row<N>(ldv, sl.lamd);
                float bl = 0.f, bld = 0.f;                    // (Bbar' lam)[c], (Bbar' lamd)[c]
#pragma unroll
                for (int i = 0; i < N; ++i) {
                    dB[i] = fmaf(g_c, fmaf(lv[i], udc, ldv[i] * uc), dB[i]);
                    bl = fmaf(bcol[i], lv[i], bl);
                    bld = fmaf(bcol[i], ldv[i], bld);
                }
                d_gb = fmaf(-tt * g_c, fmaf(udc, bl, uc * bld), d_gb);
            }
            float qx = 0.f, qxd = 0.f;
            if (s >= 1) {                                     // Q_0 = 0: no state cost at s = 0
                const float e_c = __expf(-ts * gq_c);
                sl.gq[c] = e_c;
                __syncwarp();
                float ev[N];
                load_row<N>(ev, sl.gq);
#pragma unroll
                for (int i = 0; i < N; ++i) {
                    dQ[i] = fmaf(0.5f * ev[i] * e_c, fmaf(xv[i], xdc, xdv[i] * xc), dQ[i]);
                    xv[i] *= ev[i];
                    xdv[i] *= ev[i];
                }
                qx = e_c * dot_row<N>(sl.Qb + c * LD, xv);    // (Q_s x_s)[c], (Q_s xd_s)[c]
                qxd = e_c * dot_row<N>(sl.Qb + c * LD, xdv);
                d_gq = fmaf(-ts, fmaf(xc, qxd, xdc * qx), d_gq);
            }
            if (s == 0)
                lamd_c = a_c * lamd_c;                        // lamd_0 = A_1' lamd_1 (Q_0 = 0, xd_0 = 0): the gradient of h_0
        }
        d_ri /= ri_c * ri_c;
        // ---- outputs; contraction of the three matrices with the bases
        const float qn = quiet_nan();
        if (active) {
            if (q.d_sa) q.d_sa[inst * N + c] = failed ? qn : d_sa;
            if (q.d_ga) q.d_ga[inst * N + c] = failed ? qn : d_ga;
            if (q.d_gb) q.d_gb[inst * N + c] = failed ? qn : d_gb;
            if (q.d_gq) q.d_gq[inst * N + c] = failed ? qn : d_gq;
            if (q.d_ri) q.d_ri[inst * N + c] = failed ? qn : d_ri;
            if (q.d_h0) q.d_h0[inst * N + c] = failed ? qn : lamd_c;
            if (q.GB) {
#pragma unroll
                for (int i = 0; i < N; ++i) {
                    q.GB[(inst * N + i) * (long long)N + c] = dB[i];
                    q.GQ[(inst * N + i) * (long long)N + c] = dQ[i];
                    q.GF[(inst * N + i) * (long long)N + c] = dF[i];
                }
            }
        }
        if (q.d_sb || q.d_sq || q.d_sqf) {
#pragma unroll 1
            for (int k = 0; k < r; ++k) {
                const float* Bk = p.B_basis + (long long)k * N * N + c;
                const float* Qk = p.Q_basis + (long long)k * N * N + c;
                float pb = 0.f, pq = 0.f, pf = 0.f;
#pragma unroll
                for (int i = 0; i < N; ++i) {
                    const float qv = __ldg(Qk + i * N);
                    pb = fmaf(dB[i], __ldg(Bk + i * N), pb);
                    pq = fmaf(dQ[i], qv, pq);
                    pf = fmaf(dF[i], qv, pf);
                }
                pb = seg_sum<N>(pb);
                pq = seg_sum<N>(pq);
                pf = seg_sum<N>(pf);
                if (active && c == 0) {
                    if (q.d_sb) q.d_sb[inst * r + k] = failed ? qn : pb;
                    if (q.d_sq) q.d_sq[inst * r + k] = failed ? qn : pq;
                    if (q.d_sqf) q.d_sqf[inst * r + k] = failed ? qn : pf;
                }
            }
        }
    }
}

} // namespace lgrad
} // namespace ttc
