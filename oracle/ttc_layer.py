"""Float64 oracle of one Test-Time Control layer evaluation with contextualised parameters.

TEST INFRASTRUCTURE ONLY: used by the tests, the smoke check and the benchmark's CPU-baseline
leg.  It imports nothing from the CUDA package and the CUDA package imports nothing from here.

What it computes, in the paper's notation and order:

* Contextualization paragraph of the TTC-Net section.  Given the outputs of the coefficient layers
  for one (token, head) -- ``s_A, s_GammaA, s_GammaB, s_GammaQ`` (vectors of length d), ``s_B, s_Q,
  s_Qf`` (vectors of length r), ``s_R`` -- and the shared basis matrices ``B^(i), Q^(i)``
  (i = 1..r), the LQR parameters of the planning horizon t = 1..T are

      Gamma_X = exp(-diag(s_GammaX)),                       X in {A, B, Q}
      A_t = I + Gamma_A^t diag(s_A)
      B_t = (sum_i s_B[i] B^(i)) Gamma_B^t
      Q_t = Gamma_Q^t (sum_i s_Q[i] Q^(i)) Gamma_Q^t,       Q_T overridden by sum_i s_Qf[i] Q^(i)
      R_t = diag(s_R)

* Parameterization paragraph: the powers are evaluated in the log domain, Gamma_X^t =
  exp(-t * s_GammaX), and the layer is handed the diagonal of R^{-1} (``r_inv``), not R.

* Problem statement (LQR section and Definition A.1 with zero affine terms): dynamics
  h_t = A_t h_{t-1} + B_t u_t for t = 1..T, cost sum_{t=1..T} h_t'Q_t h_t + u_t'R_t u_t, Q_0 = 0;
  the layer's output is the first optimal control u_1*.

The recursion itself is the time-varying oracle (``lqr_oracle.solve_tv``: Prop. A.1 / Alg. 1); this
module only builds the parameter sequences and maps the paper's indices to that routine's:
step s = t - 1 of the routine uses A_{s+1}, B_{s+1}, R_{s+1} and the state weight Q_s, its terminal
weight is Q_T.
"""
from __future__ import annotations

import numpy as np

from . import lqr_oracle as _lqr


def synthesize(s_a, s_ga, s_gb, s_gq, s_b, s_q, s_qf, r_inv, B_basis, Q_basis, T):
    """Parameter sequences of one (token, head) in the paper's indexing.

    Returns ``A, B, R`` of shape ``[T + 1, d, d]`` whose entry t (1 <= t <= T) is A_t, B_t, R_t (entry 0 is
    unused and left zero) and ``Q`` of shape ``[T + 1, d, d]`` with Q_0 = 0 and Q_T the override."""
    s_a, s_ga, s_gb, s_gq = (np.asarray(v, dtype=np.float64) for v in (s_a, s_ga, s_gb, s_gq))
    s_b, s_q, s_qf = (np.asarray(v, dtype=np.float64) for v in (s_b, s_q, s_qf))
    r_inv = np.asarray(r_inv, dtype=np.float64)
    B_basis = np.asarray(B_basis, dtype=np.float64)
    Q_basis = np.asarray(Q_basis, dtype=np.float64)
    d = s_a.shape[0]
    Bbar = np.einsum("i,ijk->jk", s_b, B_basis)
    Qbar = np.einsum("i,ijk->jk", s_q, Q_basis)
    Qfin = np.einsum("i,ijk->jk", s_qf, Q_basis)
    A = np.zeros((T + 1, d, d))
    B = np.zeros((T + 1, d, d))
    R = np.zeros((T + 1, d, d))
    Q = np.zeros((T + 1, d, d))
    for t in range(1, T + 1):
        gam_a = np.exp(-t * s_ga)
        gam_b = np.exp(-t * s_gb)
        gam_q = np.exp(-t * s_gq)
        A[t] = np.eye(d) + np.diag(gam_a * s_a)
        B[t] = Bbar @ np.diag(gam_b)
        R[t] = np.diag(1.0 / r_inv)
        Q[t] = np.diag(gam_q) @ Qbar @ np.diag(gam_q)
    Q[T] = Qfin
    return A, B, Q, R


def solve(s_a, s_ga, s_gb, s_gq, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis, T):
    """One layer evaluation.  Returns ``u1`` (the output u_1*), ``P0`` (value matrix at t = 0 with Q_0 = 0:
    the optimal cost is h0' P0 h0), the optimal trajectory ``h`` [T + 1, d] (h[0] = h0) and ``u`` [T, d]
    (u[t - 1] = u_t*), and ``info``."""
    A, B, Q, R = synthesize(s_a, s_ga, s_gb, s_gq, s_b, s_q, s_qf, r_inv, B_basis, Q_basis, T)
    K, P, x, u, info = _lqr.solve_tv(A[1:], B[1:], Q[:T], R[1:], Q[T], np.asarray(h0, dtype=np.float64), T)
    return dict(u1=u[0], P0=P[0], h=x, u=u, info=info)


def solve_batch(s_a, s_ga, s_gb, s_gq, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis, T, nthreads=0):
    """Many (token, head) instances: every per-instance argument has a leading instance axis.
    Returns ``u1 [N, d]``, ``P0 [N, d, d]``, ``info [N]`` and ``threads``."""
    s_a = np.asarray(s_a, dtype=np.float64)
    N, d = s_a.shape
    A = np.empty((N, T, d, d))
    B = np.empty((N, T, d, d))
    Q = np.empty((N, T, d, d))
    R = np.empty((N, T, d, d))
    Qf = np.empty((N, d, d))
    for i in range(N):
        Ai, Bi, Qi, Ri = synthesize(s_a[i], s_ga[i], s_gb[i], s_gq[i], s_b[i], s_q[i], s_qf[i], r_inv[i],
                                    B_basis, Q_basis, T)
        A[i], B[i], Q[i], R[i], Qf[i] = Ai[1:], Bi[1:], Qi[:T], Ri[1:], Qi[T]
    out = _lqr.solve_batch_tv(A, B, Q, R, Qf, np.asarray(h0, dtype=np.float64), T, (N,), first_only=True,
                              nthreads=nthreads, want=("P", "u"))
    return dict(u1=out["u"], P0=out["P"], info=out["info"], threads=out["threads"])
