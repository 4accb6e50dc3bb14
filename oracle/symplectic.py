"""float64 numpy statements of the paper's symplectic (Hamiltonian) formulation.

TEST INFRASTRUCTURE ONLY (same rule as ``lqr_oracle.c``): nothing here is used by
the CUDA path.

Contents, each in the paper's notation (paper indexing: ``h_t = A_t h_{t-1} + B_t u_t``,
``t = 1..T``, ``Q_0 = 0``):

* ``J_matrix``            -- the standard symplectic form (Lemma A.4).
* ``S_matrix``            -- forward transition ``S_t`` of ``[h; lambda]`` (Thm A.2).
* ``Sigma_matrix``        -- ``Sigma_t = (S_t^{-1})'`` as printed in Thm 3.3 / A.3.
* ``reverse_symplectic``  -- the reverse product ``[Y1 Y2] = [I Q_T] Sigma_T ... Sigma_1``
                             and ``lambda_0``, ``u_1`` (Thm A.3, first loop of Alg. 3),
                             no affine term.
* ``forward_symplectic``  -- second loop of Alg. 3: ``[h_t; lambda_t] = S_t [h_{t-1}; lambda_{t-1}]``
                             and ``u_t = -R^{-1} B' lambda_t``.
* ``costates``            -- Alg. 2 (backward co-state scan from a trajectory).
* ``pair_*``              -- the inverse-free representation of a symplectic transition
                             by the triple ``e = (A, C, J)`` with ``M(e) = S(A, G=C, Q_prev=J)``;
                             ``pair_combine`` is the block algebra of ``M(e2) M(e1)`` and
                             ``pair_apply`` the induced map on value matrices.
"""
from __future__ import annotations

import numpy as np


def J_matrix(d):
    Z, I = np.zeros((d, d)), np.eye(d)
    return np.block([[Z, I], [-I, Z]])


def S_matrix(A, B, Qprev, R):
    """Thm A.2: ``S_t`` built from ``A_t, B_t, Q_{t-1}, R_t``."""
    G = B @ np.linalg.solve(R, B.T)
    AinvT = np.linalg.inv(A.T)
    return np.block([[A + G @ AinvT @ Qprev, -G @ AinvT], [-AinvT @ Qprev, AinvT]])


def Sigma_matrix(A, B, Qprev, R):
    """Thm 3.3 / A.3: ``Sigma_t`` built from ``A_t, B_t, Q_{t-1}, R_t``."""
    G = B @ np.linalg.solve(R, B.T)
    AinvT = np.linalg.inv(A.T)
    return np.block([[AinvT, AinvT @ Qprev], [G @ AinvT, A + G @ AinvT @ Qprev]])


def reverse_symplectic(As, Bs, Qs, Rs, h0):
    """Alg. 3, reverse loop (``r_t = 0``).  ``As[t-1] = A_t`` etc. for ``t = 1..T``;
    ``Qs`` has ``T+1`` entries ``Q_0..Q_T`` (the paper sets ``Q_0 = 0``).

    Returns ``(Y1, Y2, lambda0, u1)``; ``Y1^{-1} Y2`` is the paper's value matrix at 0.
    """
    T = len(As)
    d = As[0].shape[0]
    Y = np.hstack([np.eye(d), Qs[T]])
    for t in range(T, 0, -1):
        Y = Y @ Sigma_matrix(As[t - 1], Bs[t - 1], Qs[t - 1], Rs[t - 1])
    Y1, Y2 = Y[:, :d], Y[:, d:]
    lam0 = np.linalg.solve(Y1, Y2 @ h0)
    u1 = -np.linalg.solve(Rs[0], Bs[0].T @ np.linalg.solve(As[0].T, lam0))
    return Y1, Y2, lam0, u1


def forward_symplectic(As, Bs, Qs, Rs, h0, lam0):
    """Alg. 3, forward loop.  Returns ``(h [T+1,d], lam [T+1,d], u [T,m])`` with
    ``h[0] = h0`` and ``u[t-1] = u_t``."""
    T = len(As)
    h, lam, us = [np.asarray(h0, float)], [np.asarray(lam0, float)], []
    for t in range(1, T + 1):
        z = S_matrix(As[t - 1], Bs[t - 1], Qs[t - 1], Rs[t - 1]) @ np.concatenate([h[-1], lam[-1]])
        d = len(h0)
        h.append(z[:d])
        lam.append(z[d:])
        us.append(-np.linalg.solve(Rs[t - 1], Bs[t - 1].T @ lam[-1]))
    return np.array(h), np.array(lam), np.array(us)


def costates(As, Qs, h):
    """Alg. 2: ``lambda_T = Q_T h_T``; ``lambda_t = Q_t h_t + A_{t+1}' lambda_{t+1}``;
    ``lambda_0 = A_1' lambda_1``.  ``h`` has rows ``h_0..h_T``."""
    T = len(As)
    lam = [None] * (T + 1)
    lam[T] = Qs[T] @ h[T]
    for t in range(T - 1, 0, -1):
        lam[t] = Qs[t] @ h[t] + As[t].T @ lam[t + 1]
    lam[0] = As[0].T @ lam[1]
    return np.array(lam)


# ---- inverse-free pair representation -------------------------------------------------

def pair_from_step(A, B, Q, R):
    """Element of one step: ``(A, C = B R^{-1} B', J = Q)``; ``M(e) = S(A, G=C, Q_prev=J)``."""
    return (np.array(A, float), B @ np.linalg.solve(R, B.T), np.array(Q, float))


def pair_terminal(Q):
    """Terminal element ``(0, 0, Q)``: applying anything after it leaves ``J = Q``."""
    d = Q.shape[0]
    return (np.zeros((d, d)), np.zeros((d, d)), np.array(Q, float))


def pair_to_matrix(e):
    """``M(e)`` (needs ``A`` invertible; used only to test ``M' J M = J`` and the
    product rule)."""
    A, C, Jm = e
    AinvT = np.linalg.inv(A.T)
    return np.block([[A + C @ AinvT @ Jm, -C @ AinvT], [-AinvT @ Jm, AinvT]])


def pair_combine(e1, e2):
    """``e1`` acts first (earlier in time), ``e2`` second: ``M(e1 o e2) = M(e2) M(e1)``."""
    A1, C1, J1 = e1
    A2, C2, J2 = e2
    d = A1.shape[0]
    W = np.linalg.inv(np.eye(d) + C1 @ J2)
    A12 = A2 @ W @ A1
    C12 = A2 @ W @ C1 @ A2.T + C2
    J12 = A1.T @ np.linalg.solve(np.eye(d) + J2 @ C1, J2 @ A1) + J1
    return (A12, 0.5 * (C12 + C12.T), 0.5 * (J12 + J12.T))


def pair_apply(e, P):
    """Value-matrix map of an element: ``P -> J + A' (I + P C)^{-1} P A`` (the ``J`` part
    of ``e o (0, 0, P)``).  For a one-step element this is the Riccati step."""
    A, C, Jm = e
    d = A.shape[0]
    Pn = Jm + A.T @ np.linalg.solve(np.eye(d) + P @ C, P @ A)
    return 0.5 * (Pn + Pn.T)
