"""Ties between the Riccati oracle and the paper's symplectic formulation (CPU only).

* Lemma A.4: S_t is symplectic (S'JS = J, -J S' J = S^{-1}, three block conditions);
  Sigma_t = (S_t^{-1})' equals the matrix printed in Thm 3.3.
* Thm 3.3 / A.3: Y1^{-1} Y2 of the reverse product equals the Riccati value matrix at 0
  (paper indexing, Q_0 = 0, i.e. library P_0 - Q), lambda_0 and u_1 match.
* Thm A.2 / Alg. 3 forward loop and Alg. 2 reproduce states, co-states and actions.
* Row scaling of [Y1 Y2] leaves Y1^{-1} Y2 unchanged (the normalisation of Alg. 4).
* The inverse-free pair (A, C, J): M(e) symplectic, M(e1 o e2) = M(e2) M(e1), associativity,
  apply == Riccati step, doubling/suffix powers reproduce every P_t.
These use well-conditioned A (near identity, as the paper's parameterisation keeps it) because
the Sigma products need A^{-1}.
"""
import numpy as np
import pytest

from oracle import lqr_oracle as orc
from oracle import symplectic as sp


def rand_sys(rng, n, m, near_identity=True):
    if near_identity:
        A = np.eye(n) + 0.2 * rng.standard_normal((n, n)) / np.sqrt(n)
    else:
        G = rng.standard_normal((n, n))
        A = G * 0.9 / np.max(np.abs(np.linalg.eigvals(G)))
    B = rng.standard_normal((n, m)) / np.sqrt(n)
    L = rng.standard_normal((n, n))
    Q = L @ L.T / n + 0.1 * np.eye(n)
    M = rng.standard_normal((m, m))
    R = M @ M.T / m + 0.1 * np.eye(m)
    return A, B, Q, R, rng.standard_normal(n)


@pytest.mark.parametrize("n,m", [(1, 1), (3, 2), (6, 6), (8, 5)])
def test_lemma_symplectic_and_sigma(n, m):
    rng = np.random.default_rng(n * 10 + m)
    A, B, Q, R, _ = rand_sys(rng, n, m)
    S = sp.S_matrix(A, B, Q, R)
    J = sp.J_matrix(n)
    np.testing.assert_allclose(S.T @ J @ S, J, atol=1e-11)
    np.testing.assert_allclose(-J @ S.T @ J, np.linalg.inv(S), atol=1e-10)
    As, Bs, Cs, Ds = S[:n, :n], S[:n, n:], S[n:, :n], S[n:, n:]
    np.testing.assert_allclose(As.T @ Cs, Cs.T @ As, atol=1e-11)
    np.testing.assert_allclose(Bs.T @ Ds, Ds.T @ Bs, atol=1e-11)
    np.testing.assert_allclose(As.T @ Ds - Cs.T @ Bs, np.eye(n), atol=1e-11)
    np.testing.assert_allclose(sp.Sigma_matrix(A, B, Q, R), np.linalg.inv(S).T, atol=1e-10)
    # products of symplectic matrices stay symplectic
    S2 = sp.S_matrix(A, B, np.zeros((n, n)), R)
    Pm = S @ S @ S2
    np.testing.assert_allclose(Pm.T @ J @ Pm, J, atol=1e-9)


@pytest.mark.parametrize("n,m,H", [(2, 2, 3), (4, 3, 5), (6, 6, 7)])
def test_reverse_symplectic_equals_riccati(n, m, H):
    rng = np.random.default_rng(n + m + H)
    A, B, Q, R, x0 = rand_sys(rng, n, m)
    K, P, x, u, info = orc.solve(A, B, Q, R, x0, H)
    assert info == 0
    Z = np.zeros((n, n))
    As, Bs, Rs = [A] * H, [B] * H, [R] * H
    Qs = [Z] + [Q] * H                       # Q_0 = 0, Q_1..Q_T = Q
    Y1, Y2, lam0, u1 = sp.reverse_symplectic(As, Bs, Qs, Rs, x0)
    P0_paper = np.linalg.solve(Y1, Y2)
    np.testing.assert_allclose(P0_paper, P[0] - Q, atol=1e-9)
    np.testing.assert_allclose(u1, u[0], atol=1e-9)
    np.testing.assert_allclose(lam0, (P[0] - Q) @ x0, atol=1e-9)
    # row scaling invariance (Alg. 4's normalisation)
    D = np.diag(1.0 / np.maximum(np.abs(Y1).sum(1), np.abs(Y2).sum(1)))
    np.testing.assert_allclose(np.linalg.solve(D @ Y1, D @ Y2), P0_paper, atol=1e-9)
    # forward symplectic iteration and the co-state scan give the same trajectory
    h, lam, us = sp.forward_symplectic(As, Bs, Qs, Rs, x0, lam0)
    np.testing.assert_allclose(h, x, atol=1e-7)
    np.testing.assert_allclose(us, u, atol=1e-7)
    lam2 = sp.costates(As, Qs, x)
    np.testing.assert_allclose(lam, lam2, atol=1e-7)
    # co-state = value matrix times state (paper's P_t for t>=1 is the library's)
    for t in range(1, H + 1):
        np.testing.assert_allclose(lam2[t], P[t] @ x[t], atol=1e-9)


@pytest.mark.parametrize("n,m", [(3, 2), (6, 6)])
def test_pair_algebra(n, m):
    rng = np.random.default_rng(n)
    els = [sp.pair_from_step(*rand_sys(rng, n, m)[:4]) for _ in range(3)]
    J = sp.J_matrix(n)
    for e in els:
        M = sp.pair_to_matrix(e)
        np.testing.assert_allclose(M.T @ J @ M, J, atol=1e-10)
    e12 = sp.pair_combine(els[0], els[1])
    np.testing.assert_allclose(sp.pair_to_matrix(e12), sp.pair_to_matrix(els[1]) @ sp.pair_to_matrix(els[0]), atol=1e-9)
    a = sp.pair_combine(e12, els[2])
    b = sp.pair_combine(els[0], sp.pair_combine(els[1], els[2]))
    for xa, xb in zip(a, b):
        np.testing.assert_allclose(xa, xb, atol=1e-10)
    # apply distributes over combine
    P = sp.pair_from_step(*rand_sys(rng, n, m)[:4])[2]
    np.testing.assert_allclose(sp.pair_apply(e12, P), sp.pair_apply(els[0], sp.pair_apply(els[1], P)), atol=1e-10)
    # terminal element: J part of e o (0,0,P) is apply(e, P)
    np.testing.assert_allclose(sp.pair_combine(els[0], sp.pair_terminal(P))[2], sp.pair_apply(els[0], P), atol=1e-11)


@pytest.mark.parametrize("n,m,H,ni", [(4, 4, 8, True), (8, 8, 13, False), (16, 16, 16, False), (6, 3, 7, False)])
def test_pair_powers_reproduce_riccati(n, m, H, ni):
    rng = np.random.default_rng(H)
    A, B, Q, R, x0 = rand_sys(rng, n, m, near_identity=ni)
    K, P, x, u, info = orc.solve(A, B, Q, R, x0, H)
    e = sp.pair_from_step(A, B, Q, R)
    # one application == one Riccati step
    np.testing.assert_allclose(sp.pair_apply(e, Q), P[H - 1], atol=1e-11)
    # doubling schedule: after round r, e^(2^r) applied to P_{H-k+2^r} gives P_{H-k}
    Ps = {H: Q}
    ep, step = e, 1
    while step <= H:
        for k in range(step, min(2 * step, H + 1)):
            Ps[H - k] = sp.pair_apply(ep, Ps[H - k + step])
        ep = sp.pair_combine(ep, ep)
        step *= 2
    for t in range(H + 1):
        np.testing.assert_allclose(Ps[t], P[t], rtol=0, atol=1e-10 * np.max(np.abs(P[0])))
