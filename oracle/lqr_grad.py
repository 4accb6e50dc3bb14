"""Float64 oracle of the gradients of a Test-Time Control layer's output (Thm 3.2: primal and dual LQR).

TEST INFRASTRUCTURE ONLY: used by the tests, the smoke check and the benchmark's CPU-baseline
leg.  It imports nothing from the CUDA package and the CUDA package imports nothing from here.

The layer's output is the first optimal control ``o = u_0*`` of the time-varying problem

    minimise  1/2 sum_{t<H} (x_t'Q_t x_t + u_t'R_t u_t) + 1/2 x_H'Qf x_H,    x_{t+1} = A_t x_t + B_t u_t

(library indexing; with the paper's ``h_t = A_t h_{t-1} + B_t u_t``, t = 1..T: ``x_t = h_t``, ``A_t(here) =
A_{t+1}(paper)``, likewise B, R and u; ``Q_t(here) = Q_t(paper)``, ``Qf = Q_T``).  Given ``g = dl/do`` for a scalar
loss ``l(o)``, Thm 3.2 gives the gradients with respect to every parameter matrix and the initial state from the
solutions of two KKT systems, in the paper's order:

1. primal LQR: states ``x_t``, controls ``u_t`` (Prop. A.1 / Alg. 1: the pinned time-varying routine);
2. co-states by the backward relation stated before Thm 3.2 (stationarity of the Lagrangian in ``h_t``):
   ``lam_H = Qf x_H``, ``lam_t = A_t' lam_{t+1} + Q_t x_t``;
3. dual LQR: the same matrices, zero initial state and the extra cost ``g'u_0`` on the first control (Prop. A.1 with
   the linear control cost ``r_0 = g``, ``r_t = 0`` otherwise: the pinned affine routine), giving ``xd_t``, ``ud_t``
   and, by the same backward relation, ``lamd_t``;
4. the outer products of Thm 3.2, re-indexed:
       dA_t = lam_{t+1} xd_t' + lamd_{t+1} x_t'        dB_t = lam_{t+1} ud_t' + lamd_{t+1} u_t'
       dQ_t = 1/2 (x_t xd_t' + xd_t x_t')  (t <= H-1; dQf the same at t = H)
       dR_t = 1/2 (u_t ud_t' + ud_t u_t')              dx0 = lamd_0 .

The gradients with respect to Q_t, R_t are those of the theorem: symmetric, i.e. the derivative along symmetric
perturbations of the weights.
"""
from __future__ import annotations

import numpy as np

from . import lqr_oracle as _lqr


def _at(M, t):
    return M[t] if M.ndim == 3 else M


def costates(A, Q, Qf, x, H):
    """lam_H = Qf x_H ; lam_t = A_t' lam_{t+1} + Q_t x_t  (t = H-1..0)."""
    n = x.shape[1]
    lam = np.zeros((H + 1, n))
    lam[H] = Qf @ x[H]
    for t in range(H - 1, -1, -1):
        lam[t] = _at(A, t).T @ lam[t + 1] + _at(Q, t) @ x[t]
    return lam


def grad(A, B, Q, R, Qf, x0, g, H):
    """Gradients of ``l(u_0*)`` given ``g = dl/du_0*``.  ``A [H,n,n]`` or ``[n,n]`` (constant in time), likewise
    ``B, Q, R``; the gradients are always returned per time step (for a constant matrix the caller sums over t).

    Returns a dict: ``dA [H,n,n]``, ``dB [H,n,m]``, ``dQ [H,n,n]``, ``dQf [n,n]``, ``dR [H,m,m]``, ``dx0 [n]``, the
    forward output ``u0 [m]``, the two KKT solutions (``x, u, lam, xd, ud, lamd``) and ``info``."""
    A, B, Q, R, Qf, x0, g = (np.asarray(v, dtype=np.float64) for v in (A, B, Q, R, Qf, x0, g))
    n, m = B.shape[-2:]
    K, P, x, u, info = _lqr.solve_tv(A, B, Q, R, Qf, x0, H)
    lam = costates(A, Q, Qf, x, H)
    r = np.zeros((H, m))
    r[0] = g
    dual = _lqr.solve_affine(A, B, Q, R, r, Qf, np.zeros(n), H)
    xd, ud = dual["x"], dual["u"]
    lamd = costates(A, Q, Qf, xd, H)
    dA = np.empty((H, n, n)); dB = np.empty((H, n, m)); dQ = np.empty((H, n, n)); dR = np.empty((H, m, m))
    for t in range(H):
        dA[t] = np.outer(lam[t + 1], xd[t]) + np.outer(lamd[t + 1], x[t])
        dB[t] = np.outer(lam[t + 1], ud[t]) + np.outer(lamd[t + 1], u[t])
        dQ[t] = 0.5 * (np.outer(x[t], xd[t]) + np.outer(xd[t], x[t]))
        dR[t] = 0.5 * (np.outer(u[t], ud[t]) + np.outer(ud[t], u[t]))
    dQf = 0.5 * (np.outer(x[H], xd[H]) + np.outer(xd[H], x[H]))
    return dict(dA=dA, dB=dB, dQ=dQ, dQf=dQf, dR=dR, dx0=lamd[0].copy(), u0=u[0].copy(),
                x=x, u=u, lam=lam, xd=xd, ud=ud, lamd=lamd, info=int(info) | int(dual["info"]))
