"""Float64 oracle of the gradients of one contextualised Test-Time Control layer evaluation with respect to
what the coefficient layers hand over (Thm 3.2 followed by the chain rule through the Contextualization and
Parameterization paragraphs of the TTC-Net section).

TEST INFRASTRUCTURE ONLY: used by the tests, the smoke check and the benchmark's CPU-baseline
leg.  It imports nothing from the CUDA package and the CUDA package imports nothing from here.

Steps, in the paper's order:

1. ``ttc_layer.synthesize`` builds A_t, B_t, Q_t, R_t (t = 1..T, Q_0 = 0, Q_T overridden) from the coefficients;
2. ``lqr_grad.grad`` (Thm 3.2: primal and dual LQR, co-states, outer products) gives the gradient of a scalar loss
   l(u_1*) with respect to every A_t, B_t, Q_t, R_t, Q_T and h_0, given g = dl/du_1*;
3. the chain rule through step 1, written out term by term:
       A_t = I + diag(e^{-t gA} sA)        ->  d sA[i]  = sum_t e^{-t gA_i} dA_t[i,i]
                                               d gA[i]  = sum_t -t e^{-t gA_i} sA[i] dA_t[i,i]
       B_t = Bbar diag(e^{-t gB})           ->  d Bbar   = sum_t dB_t diag(e^{-t gB})
                                               d gB[j]  = sum_t -t e^{-t gB_j} sum_i dB_t[i,j] Bbar[i,j]
       Q_t = G_t Qbar G_t, G_t = diag(e^{-t gQ}), 1 <= t <= T-1
                                           ->  d Qbar   = sum_t G_t dQ_t G_t
                                               d gQ[i]  = sum_t -2 t sum_j dQ_t[i,j] Q_t[i,j]        (dQ_t symmetric)
       Q_T = Qfin                           ->  d Qfin   = dQ_T
       R_t = diag(1 / r_inv)                ->  d r_inv[j] = -sum_t dR_t[j,j] / r_inv[j]^2
       Bbar = sum_k sB[k] B^(k)             ->  d sB[k] = <d Bbar, B^(k)>,   d B^(k) = sB[k] d Bbar
       Qbar, Qfin = sum_k sQ[k], sQf[k] Q^(k) -> d sQ[k] = <d Qbar, Q^(k)>, d sQf[k] = <d Qfin, Q^(k)>,
                                               d Q^(k) = sQ[k] d Qbar + sQf[k] d Qfin
   (the basis gradients are those of ONE instance; a caller sums them over the instances that share the bases).
"""
from __future__ import annotations

import numpy as np

from . import lqr_grad as _grad
from . import ttc_layer as _layer


def grad(s_a, s_ga, s_gb, s_gq, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis, T, g):
    """Gradients of ``l(u_1*)`` given ``g = dl/du_1*`` for one (token, head).  Returns a dict with ``s_a, s_gamma_a,
    s_gamma_b, s_gamma_q, r_inv, h0`` (length d), ``s_b, s_q, s_qf`` (length r), ``B_basis, Q_basis`` ([r, d, d]),
    the forward output ``u1`` and ``info``."""
    s_a, s_ga, s_gb, s_gq, r_inv, h0, g = (np.asarray(v, dtype=np.float64) for v in (s_a, s_ga, s_gb, s_gq, r_inv, h0, g))
    s_b, s_q, s_qf = (np.asarray(v, dtype=np.float64) for v in (s_b, s_q, s_qf))
    B_basis = np.asarray(B_basis, dtype=np.float64)
    Q_basis = np.asarray(Q_basis, dtype=np.float64)
    d = s_a.shape[0]
    A, B, Q, R = _layer.synthesize(s_a, s_ga, s_gb, s_gq, s_b, s_q, s_qf, r_inv, B_basis, Q_basis, T)
    # the dense routine's step s = t - 1 uses A_{s+1}, B_{s+1}, R_{s+1} and the state weight Q_s; terminal weight Q_T
    dense = _grad.grad(A[1:], B[1:], Q[:T], R[1:], Q[T], h0, g, T)
    Bbar = np.einsum("i,ijk->jk", s_b, B_basis)
    d_sa, d_ga, d_gb, d_gq, d_ri = (np.zeros(d) for _ in range(5))
    d_Bbar, d_Qbar = np.zeros((d, d)), np.zeros((d, d))
    for t in range(1, T + 1):
        dA, dB, dR = dense["dA"][t - 1], dense["dB"][t - 1], dense["dR"][t - 1]
        ea, eb = np.exp(-t * s_ga), np.exp(-t * s_gb)
        d_sa += ea * np.diag(dA)
        d_ga += -t * ea * s_a * np.diag(dA)
        d_Bbar += dB * eb[None, :]
        d_gb += -t * eb * np.sum(dB * Bbar, axis=0)
        d_ri += -np.diag(dR) / r_inv ** 2
    for t in range(1, T):                       # Q_0 = 0 and Q_T is the override: neither depends on Qbar, gQ
        dQ = dense["dQ"][t]
        eq = np.exp(-t * s_gq)
        d_Qbar += eq[:, None] * dQ * eq[None, :]
        d_gq += -2.0 * t * np.sum(dQ * Q[t], axis=1)
    d_Qfin = dense["dQf"]
    return dict(
        s_a=d_sa, s_gamma_a=d_ga, s_gamma_b=d_gb, s_gamma_q=d_gq, r_inv=d_ri, h0=dense["dx0"],
        s_b=np.einsum("jk,ijk->i", d_Bbar, B_basis), s_q=np.einsum("jk,ijk->i", d_Qbar, Q_basis),
        s_qf=np.einsum("jk,ijk->i", d_Qfin, Q_basis),
        B_basis=s_b[:, None, None] * d_Bbar[None], Q_basis=s_q[:, None, None] * d_Qbar[None] + s_qf[:, None, None] * d_Qfin[None],
        u1=dense["u0"], info=dense["info"])
