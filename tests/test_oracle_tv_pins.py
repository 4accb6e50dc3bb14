"""Pins of the time-varying oracle (A_t, B_t, Q_t, R_t, terminal weight Q_f) against things other than itself.

* the stacked KKT system of the time-varying finite-horizon QP (Definition A.1 written as one dense linear system,
  the matrix form used in the proof of Thm 3.2), solved with a general dense solver: trajectory, cost, and -- through
  tail problems started at t from unit vectors -- every K_t and P_t;
* with equal matrices at every t and Q_f = Q it must reproduce the time-invariant function bit for bit;
* a hand-rolled scalar case whose stage data differ per step, checked against exact rational arithmetic;
* the cost identity J(rollout) = x_0'P_0 x_0 and optimality under perturbation of the controls;
* a time shift: the tail of a problem is the problem of the tail.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import lqr_oracle as orc


def rand_tv(rng, n, m, H):
    A = np.stack([rng.standard_normal((n, n)) * 0.6 / np.sqrt(n) + 0.3 * np.eye(n) for _ in range(H)])
    B = rng.standard_normal((H, n, m)) / np.sqrt(n)
    Q = np.stack([(lambda L: L @ L.T / n + 0.1 * np.eye(n))(rng.standard_normal((n, n))) for _ in range(H)])
    R = np.stack([(lambda M: M @ M.T / m + 0.1 * np.eye(m))(rng.standard_normal((m, m))) for _ in range(H)])
    Lf = rng.standard_normal((n, n))
    Qf = Lf @ Lf.T / n + 0.05 * np.eye(n)
    return A, B, Q, R, Qf, rng.standard_normal(n)


def kkt_tv(A, B, Q, R, Qf, x0):
    """min sum_{t<H} x_t'Q_t x_t + u_t'R_t u_t + x_H'Q_f x_H  s.t. x_{t+1} = A_t x_t + B_t u_t, x_0 given, as ONE dense
    linear system [[C, F'], [F, 0]] [z; xi] = [0; b], z = [x_0..x_H, u_0..u_{H-1}]."""
    H, n, m = B.shape
    nz, nc, uo = (H + 1) * n + H * m, (H + 1) * n, (H + 1) * n
    C = np.zeros((nz, nz))
    for t in range(H):
        C[t * n:(t + 1) * n, t * n:(t + 1) * n] = 2 * Q[t]
        C[uo + t * m:uo + (t + 1) * m, uo + t * m:uo + (t + 1) * m] = 2 * R[t]
    C[H * n:(H + 1) * n, H * n:(H + 1) * n] = 2 * Qf
    F = np.zeros((nc, nz))
    b = np.zeros(nc)
    F[:n, :n] = -np.eye(n)
    b[:n] = -x0
    for t in range(H):
        r = (t + 1) * n
        F[r:r + n, t * n:(t + 1) * n] = A[t]
        F[r:r + n, (t + 1) * n:(t + 2) * n] = -np.eye(n)
        F[r:r + n, uo + t * m:uo + (t + 1) * m] = B[t]
    sol = np.linalg.solve(np.block([[C, F.T], [F, np.zeros((nc, nc))]]), np.concatenate([np.zeros(nz), b]))
    z = sol[:nz]
    return z[:uo].reshape(H + 1, n), z[uo:].reshape(H, m), 0.5 * z @ C @ z


@pytest.mark.parametrize("n,m,H", [(1, 1, 1), (1, 1, 5), (2, 1, 3), (3, 2, 4), (4, 3, 3), (2, 3, 2), (3, 3, 5)])
def test_bruteforce_kkt_time_varying(n, m, H):
    rng = np.random.default_rng(7 + 100 * n + 10 * m + H)
    A, B, Q, R, Qf, x0 = rand_tv(rng, n, m, H)
    K, P, x, u, info = orc.solve_tv(A, B, Q, R, Qf, x0, H)
    assert info == 0
    xb, ub, cb = kkt_tv(A, B, Q, R, Qf, x0)
    np.testing.assert_allclose(x, xb, rtol=0, atol=1e-11)
    np.testing.assert_allclose(u, ub, rtol=0, atol=1e-11)
    assert abs(x0 @ P[0] @ x0 - cb) <= 1e-11 * max(1.0, abs(cb))
    np.testing.assert_array_equal(P[H], Qf)
    I = np.eye(n)
    for t in range(H):           # K_t, P_t from the tail problem that starts at t (its own brute-force solves)
        At, Bt, Qt, Rt = A[t:], B[t:], Q[t:], R[t:]
        Kt = np.zeros((m, n))
        for j in range(n):
            Kt[:, j] = kkt_tv(At, Bt, Qt, Rt, Qf, I[j])[1][0]
        Pt = np.zeros((n, n))
        for i in range(n):
            Pt[i, i] = kkt_tv(At, Bt, Qt, Rt, Qf, I[i])[2]
        for i in range(n):
            for j in range(i + 1, n):
                Pt[i, j] = Pt[j, i] = (kkt_tv(At, Bt, Qt, Rt, Qf, I[i] + I[j])[2] - Pt[i, i] - Pt[j, j]) / 2.0
        np.testing.assert_allclose(K[t], Kt, rtol=0, atol=1e-10)
        np.testing.assert_allclose(P[t], Pt, rtol=0, atol=1e-10)


def test_equal_matrices_reduce_to_the_time_invariant_function_bitwise():
    rng = np.random.default_rng(3)
    n, m, H = 5, 3, 7
    G = rng.standard_normal((n, n))
    A = 0.9 * G / np.max(np.abs(np.linalg.eigvals(G)))
    B = rng.standard_normal((n, m))
    L = rng.standard_normal((n, n)); Q = L @ L.T + 0.1 * np.eye(n)
    M = rng.standard_normal((m, m)); R = M @ M.T + 0.1 * np.eye(m)
    x0 = rng.standard_normal(n)
    ref = orc.solve(A, B, Q, R, x0, H)
    rep = lambda a: np.repeat(a[None], H, axis=0)
    for tv in (orc.solve_tv(rep(A), rep(B), rep(Q), rep(R), Q, x0, H), orc.solve_tv(A, B, Q, R, Q, x0, H),
               orc.solve_tv(rep(A), B, Q, rep(R), Q, x0, H)):
        for a, b in zip(ref[:4], tv[:4]):
            np.testing.assert_array_equal(a, b)
        assert tv[4] == 0


def test_scalar_case_in_exact_rational_arithmetic():
    # n = m = 1, data differ per step; the recursion is carried out in exact fractions by hand
    a = [Fraction(1, 2), Fraction(3, 2), Fraction(-1), Fraction(2, 3)]
    b = [Fraction(1), Fraction(1, 3), Fraction(2), Fraction(-1, 2)]
    q = [Fraction(1), Fraction(2), Fraction(1, 4), Fraction(3)]
    r = [Fraction(1, 2), Fraction(1), Fraction(3), Fraction(1, 5)]
    qf = Fraction(5, 2)
    H = 4
    P = [None] * (H + 1)
    Kf = [None] * H
    P[H] = qf
    for t in range(H - 1, -1, -1):
        s = r[t] + b[t] * P[t + 1] * b[t]
        Kf[t] = -(b[t] * P[t + 1] * a[t]) / s
        P[t] = q[t] + a[t] * P[t + 1] * a[t] + (b[t] * P[t + 1] * a[t]) * Kf[t]
    f = lambda v: np.array([float(e) for e in v])
    K, Po, x, u, info = orc.solve_tv(f(a).reshape(H, 1, 1), f(b).reshape(H, 1, 1), f(q).reshape(H, 1, 1),
                                     f(r).reshape(H, 1, 1), np.array([[float(qf)]]), np.array([1.0]), H)
    assert info == 0
    np.testing.assert_allclose(Po[:, 0, 0], f(P), rtol=1e-14)
    np.testing.assert_allclose(K[:, 0, 0], f(Kf), rtol=1e-14)
    xs = [Fraction(1)]
    for t in range(H):
        xs.append((a[t] + b[t] * Kf[t]) * xs[-1])
    np.testing.assert_allclose(x[:, 0], f(xs), rtol=1e-13)


@pytest.mark.parametrize("n,m,H,seed", [(3, 2, 6, 0), (6, 6, 4, 1), (5, 2, 9, 2)])
def test_cost_identity_and_optimality(n, m, H, seed):
    rng = np.random.default_rng(seed)
    A, B, Q, R, Qf, x0 = rand_tv(rng, n, m, H)
    K, P, x, u, info = orc.solve_tv(A, B, Q, R, Qf, x0, H)
    assert info == 0

    def cost(us):
        xt, J = x0.copy(), 0.0
        for t in range(H):
            J += xt @ Q[t] @ xt + us[t] @ R[t] @ us[t]
            xt = A[t] @ xt + B[t] @ us[t]
        return J + xt @ Qf @ xt

    J = cost(u)
    assert abs(J - x0 @ P[0] @ x0) <= 1e-10 * max(1.0, J)
    for _ in range(10):
        assert cost(u + 1e-3 * rng.standard_normal(u.shape)) >= J - 1e-12
    for t in range(H + 1):
        np.testing.assert_allclose(P[t], P[t].T, atol=1e-12)
        assert np.linalg.eigvalsh(P[t]).min() > 0


def test_tail_of_the_problem_is_the_problem_of_the_tail_and_batch():
    rng = np.random.default_rng(11)
    n, m, H = 4, 3, 6
    A, B, Q, R, Qf, x0 = rand_tv(rng, n, m, H)
    K, P, x, u, _ = orc.solve_tv(A, B, Q, R, Qf, x0, H)
    for t in (1, 3, 5):
        Kt, Pt, xt, ut, _ = orc.solve_tv(A[t:], B[t:], Q[t:], R[t:], Qf, x[t], H - t)
        np.testing.assert_allclose(Kt, K[t:], atol=1e-12)
        np.testing.assert_allclose(Pt, P[t:], atol=1e-12)
        np.testing.assert_allclose(xt, x[t:], atol=1e-12)
    # batch front end: per-head time-varying A, B, R, per-token Q_t, Q_f, x0; mixed time-invariant operand
    S, Hd, T = 2, 2, 3
    Ab = np.stack([rand_tv(rng, n, m, H)[0] for _ in range(Hd)]).reshape(1, Hd, 1, H, n, n)
    Bb = rng.standard_normal((1, Hd, 1, n, m))                          # time-invariant B per head
    Rb = np.stack([rand_tv(rng, n, m, H)[3] for _ in range(Hd)]).reshape(1, Hd, 1, H, m, m)
    Qb = np.stack([rand_tv(rng, n, m, H)[2] for _ in range(S * Hd * T)]).reshape(S, Hd, T, H, n, n)
    Qfb = np.stack([rand_tv(rng, n, m, H)[4] for _ in range(S * Hd * T)]).reshape(S, Hd, T, n, n)
    xb = rng.standard_normal((S, Hd, T, n))
    out = orc.solve_batch_tv(Ab, Bb, Qb, Rb, Qfb, xb, H, (S, Hd, T), tv=("A", "Q", "R"))
    assert np.all(out["info"] == 0)
    i = 0
    for s in range(S):
        for h in range(Hd):
            for k in range(T):
                Kk, Pk, xk, uk, _ = orc.solve_tv(Ab[0, h, 0], Bb[0, h, 0], Qb[s, h, k], Rb[0, h, 0], Qfb[s, h, k], xb[s, h, k], H)
                np.testing.assert_array_equal(out["K"][i], Kk)
                np.testing.assert_array_equal(out["P"][i], Pk)
                np.testing.assert_array_equal(out["u"][i], uk)
                i += 1
