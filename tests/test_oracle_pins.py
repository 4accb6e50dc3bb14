"""Pins of the float64 CPU oracle against things other than itself.

Everything here runs on the CPU.  Each test ties the oracle's Riccati recursion and
rollout (Prop. 3.1, Alg. 1) to a definition, a closed form, an invariant or a library
routine that was not written from the oracle's code:

* the stacked KKT system of the finite-horizon QP (matrix form in the proof of Thm 3.2),
  solved with a general dense solver;
* the scalar case a=b=q=r=1, whose value sequence is a ratio of Fibonacci numbers;
* decoupled (diagonal) systems and an orthogonal change of basis;
* B=0, A=0, H=1, very large R;
* symmetry / definiteness / monotonicity of P_t, optimal cost x0'P0x0, optimality under
  perturbation, KKT residuals with lambda_t = P_t x_t (Eqs. of the KKT section);
* P_0 -> the DARE solution (scipy) for long horizons.
"""
from fractions import Fraction

import numpy as np
import pytest
import scipy.linalg

from oracle import lqr_oracle as orc


def rand_sys(rng, n, m, rho=0.9):
    G = rng.standard_normal((n, n))
    A = G * rho / max(np.max(np.abs(np.linalg.eigvals(G))), 1e-12)
    B = rng.standard_normal((n, m)) / np.sqrt(n)
    L = rng.standard_normal((n, n))
    Q = L @ L.T / n + 0.1 * np.eye(n)
    M = rng.standard_normal((m, m))
    R = M @ M.T / m + 0.1 * np.eye(m)
    return A, B, Q, R, rng.standard_normal(n)


def kkt_bruteforce(A, B, Q, R, x0, H):
    """Solve min sum_t x_t'Qx_t + u_t'Ru_t + x_H'Qx_H  s.t. dynamics, as ONE dense linear
    system [[C, F'], [F, 0]] [z; xi] = [0; b] with z = [x_0..x_H, u_0..u_{H-1}]."""
    n, m = B.shape
    nz = (H + 1) * n + H * m
    nc = (H + 1) * n
    C = np.zeros((nz, nz))
    for t in range(H + 1):
        C[t * n:(t + 1) * n, t * n:(t + 1) * n] = 2 * Q
    uo = (H + 1) * n
    for t in range(H):
        C[uo + t * m:uo + (t + 1) * m, uo + t * m:uo + (t + 1) * m] = 2 * R
    F = np.zeros((nc, nz))
    b = np.zeros(nc)
    F[:n, :n] = -np.eye(n)
    b[:n] = -x0
    for t in range(H):
        r = (t + 1) * n
        F[r:r + n, t * n:(t + 1) * n] = A
        F[r:r + n, (t + 1) * n:(t + 2) * n] = -np.eye(n)
        F[r:r + n, uo + t * m:uo + (t + 1) * m] = B
    KKT = np.block([[C, F.T], [F, np.zeros((nc, nc))]])
    sol = np.linalg.solve(KKT, np.concatenate([np.zeros(nz), b]))
    z = sol[:nz]
    x = z[:uo].reshape(H + 1, n)
    u = z[uo:].reshape(H, m)
    cost = 0.5 * z @ C @ z
    return x, u, cost


@pytest.mark.parametrize("n,m,H", [(1, 1, 1), (1, 1, 4), (2, 1, 3), (3, 2, 5), (4, 3, 4), (2, 3, 2), (4, 4, 5)])
def test_bruteforce_kkt_trajectory_cost_and_gains(n, m, H):
    rng = np.random.default_rng(100 * n + 10 * m + H)
    A, B, Q, R, x0 = rand_sys(rng, n, m)
    K, P, x, u, info = orc.solve(A, B, Q, R, x0, H)
    assert info == 0
    xb, ub, cb = kkt_bruteforce(A, B, Q, R, x0, H)
    np.testing.assert_allclose(x, xb, rtol=0, atol=1e-11)
    np.testing.assert_allclose(u, ub, rtol=0, atol=1e-11)
    assert abs(x0 @ P[0] @ x0 - cb) <= 1e-11 * max(1.0, abs(cb))
    # K_t and P_t of the tail problem starting at t (time-invariant: horizon H-t)
    I = np.eye(n)
    for t in range(H):
        Ht = H - t
        Kt = np.zeros((m, n))
        Jv = np.zeros((n, n))
        for j in range(n):
            _, uj, _ = kkt_bruteforce(A, B, Q, R, I[j], Ht)
            Kt[:, j] = uj[0]
        for i in range(n):
            for j in range(i, n):
                _, _, cij = kkt_bruteforce(A, B, Q, R, I[i] + I[j], Ht)
                Jv[i, j] = Jv[j, i] = cij
        Pt = np.zeros((n, n))
        for i in range(n):
            Pt[i, i] = Jv[i, i] / 4.0
        for i in range(n):
            for j in range(i + 1, n):
                Pt[i, j] = Pt[j, i] = (Jv[i, j] - Pt[i, i] - Pt[j, j]) / 2.0
        np.testing.assert_allclose(K[t], Kt, rtol=0, atol=1e-10)
        np.testing.assert_allclose(P[t], Pt, rtol=0, atol=1e-10)
    np.testing.assert_allclose(P[H], Q, rtol=0, atol=0)


def test_scalar_fibonacci_closed_form():
    # a=b=q=r=1: P_{H-k} = F_{2k+2}/F_{2k+1}, K_{H-1-k} = -P_{H-k}/(1+P_{H-k})
    H = 12
    fib = [0, 1]
    while len(fib) < 2 * H + 4:
        fib.append(fib[-1] + fib[-2])
    one = np.ones((1, 1))
    K, P, x, u, info = orc.solve(one, one, one, one, np.array([1.0]), H)
    assert info == 0
    for k in range(H + 1):
        want = Fraction(fib[2 * k + 2], fib[2 * k + 1])
        assert abs(P[H - k, 0, 0] - float(want)) < 1e-14
        if k < H:
            wk = -want / (1 + want)
            assert abs(K[H - 1 - k, 0, 0] - float(wk)) < 1e-14
    assert [Fraction(fib[2 * k + 2], fib[2 * k + 1]) for k in range(5)] == [
        Fraction(1), Fraction(3, 2), Fraction(8, 5), Fraction(21, 13), Fraction(55, 34)]
    assert abs(P[0, 0, 0] - (1 + 5 ** 0.5) / 2) < 1e-8
    # rollout: x_{t+1} = (1 + K_t) x_t, u_t = K_t x_t
    xt = 1.0
    for t in range(H):
        assert abs(u[t, 0] - K[t, 0, 0] * xt) < 1e-14
        xt = (1 + K[t, 0, 0]) * xt
        assert abs(x[t + 1, 0] - xt) < 1e-14


def scalar_recursion(a, b, q, r, H):
    P = [0.0] * (H + 1)
    K = [0.0] * H
    P[H] = q
    for t in range(H - 1, -1, -1):
        K[t] = -a * b * P[t + 1] / (r + b * b * P[t + 1])
        P[t] = q + a * a * P[t + 1] * r / (r + b * b * P[t + 1])
    return K, P


def test_decoupled_and_change_of_basis():
    rng = np.random.default_rng(7)
    n, H = 5, 9
    a = rng.uniform(-1.2, 1.2, n)
    b = rng.uniform(0.3, 1.5, n) * rng.choice([-1, 1], n)
    q = rng.uniform(0.1, 2.0, n)
    r = rng.uniform(0.1, 2.0, n)
    x0 = rng.standard_normal(n)
    K, P, x, u, info = orc.solve(np.diag(a), np.diag(b), np.diag(q), np.diag(r), x0, H)
    assert info == 0
    for i in range(n):
        Ks, Ps = scalar_recursion(a[i], b[i], q[i], r[i], H)
        np.testing.assert_allclose(P[:, i, i], Ps, rtol=1e-13)
        np.testing.assert_allclose(K[:, i, i], Ks, rtol=1e-13)
    offdiag = P - np.einsum("tii->ti", P)[:, :, None] * np.eye(n)
    assert np.max(np.abs(offdiag)) == 0.0
    # orthogonal change of basis of states (U) and controls (V)
    U, _ = np.linalg.qr(rng.standard_normal((n, n)))
    V, _ = np.linalg.qr(rng.standard_normal((n, n)))
    K2, P2, x2, u2, info2 = orc.solve(U @ np.diag(a) @ U.T, U @ np.diag(b) @ V.T, U @ np.diag(q) @ U.T,
                                      V @ np.diag(r) @ V.T, U @ x0, H)
    assert info2 == 0
    np.testing.assert_allclose(K2, V @ K @ U.T, atol=1e-12)
    np.testing.assert_allclose(P2, U @ P @ U.T, atol=1e-12)
    np.testing.assert_allclose(x2, x @ U.T, atol=1e-12)
    np.testing.assert_allclose(u2, u @ V.T, atol=1e-12)


def test_special_cases():
    rng = np.random.default_rng(11)
    n, m, H = 4, 3, 6
    A, B, Q, R, x0 = rand_sys(rng, n, m)
    # B = 0: no control authority
    K, P, x, u, info = orc.solve(A, np.zeros((n, m)), Q, R, x0, H)
    assert info == 0 and np.all(K == 0) and np.all(u == 0)
    for t in range(H + 1):
        want = sum(np.linalg.matrix_power(A.T, k) @ Q @ np.linalg.matrix_power(A, k) for k in range(H - t + 1))
        np.testing.assert_allclose(P[t], want, atol=1e-12)
        np.testing.assert_allclose(x[t], np.linalg.matrix_power(A, t) @ x0, atol=1e-12)
    # A = 0: P_t = Q for t < H too, states vanish after the first step
    K, P, x, u, info = orc.solve(np.zeros((n, n)), B, Q, R, x0, H)
    assert info == 0
    for t in range(H + 1):
        np.testing.assert_allclose(P[t], Q, atol=1e-14)
    assert np.all(K == 0) and np.all(x[1:] == 0)
    # H = 1 closed form
    K, P, x, u, info = orc.solve(A, B, Q, R, x0, 1)
    S = R + B.T @ Q @ B
    K0 = -np.linalg.solve(S, B.T @ Q @ A)
    np.testing.assert_allclose(K[0], K0, atol=1e-13)
    np.testing.assert_allclose(P[0], Q + A.T @ Q @ A - A.T @ Q @ B @ np.linalg.solve(S, B.T @ Q @ A), atol=1e-13)
    np.testing.assert_allclose(u[0], K0 @ x0, atol=1e-13)
    np.testing.assert_allclose(x[1], (A + B @ K0) @ x0, atol=1e-13)
    # R -> infinity: control switched off
    K, P, x, u, info = orc.solve(A, B, Q, 1e14 * R, x0, H)
    Kb, Pb, xb, ub, _ = orc.solve(A, np.zeros((n, m)), Q, R, x0, H)
    assert np.max(np.abs(K)) < 1e-12
    np.testing.assert_allclose(P, Pb, atol=1e-10)


@pytest.mark.parametrize("n,m,H,seed", [(6, 4, 10, 0), (8, 8, 8, 1), (16, 16, 16, 2), (5, 7, 12, 3)])
def test_invariants(n, m, H, seed):
    rng = np.random.default_rng(seed)
    A, B, Q, R, x0 = rand_sys(rng, n, m)
    K, P, x, u, info = orc.solve(A, B, Q, R, x0, H)
    assert info == 0
    for t in range(H + 1):
        assert np.array_equal(P[t], P[t].T)
        assert np.linalg.eigvalsh(P[t]).min() > 0
        if t < H:  # P_t >= P_{t+1}
            assert np.linalg.eigvalsh(P[t] - P[t + 1]).min() > -1e-11
    def cost(xs, us):
        return sum(xs[t] @ Q @ xs[t] for t in range(H + 1)) + sum(us[t] @ R @ us[t] for t in range(H))
    Jstar = cost(x, u)
    assert abs(Jstar - x0 @ P[0] @ x0) < 1e-11 * Jstar
    # cost-to-go along the trajectory: J_t = x_t' P_t x_t
    for t in range(H + 1):
        Jt = sum(x[s] @ Q @ x[s] for s in range(t, H + 1)) + sum(u[s] @ R @ u[s] for s in range(t, H))
        assert abs(Jt - x[t] @ P[t] @ x[t]) < 1e-11 * max(Jstar, 1.0)
    # any perturbed control sequence costs more
    for _ in range(20):
        du = 1e-3 * rng.standard_normal(u.shape)
        xs = [x0]
        for t in range(H):
            xs.append(A @ xs[-1] + B @ (u[t] + du[t]))
        assert cost(np.array(xs), u + du) > Jstar
    # KKT residuals with lambda_t = P_t x_t (cost without the 1/2: multipliers scale by 2,
    # so the conditions read Q x_t + A' lam_{t+1} = lam_t, R u_t + B' lam_{t+1} = 0, lam_H = Q x_H)
    lam = np.einsum("tij,tj->ti", P, x)
    np.testing.assert_allclose(lam[H], Q @ x[H], atol=1e-12)
    for t in range(H):
        np.testing.assert_allclose(Q @ x[t] + A.T @ lam[t + 1], lam[t], atol=1e-10)
        np.testing.assert_allclose(R @ u[t] + B.T @ lam[t + 1], 0, atol=1e-10)
        np.testing.assert_allclose(A @ x[t] + B @ u[t], x[t + 1], atol=1e-12)


@pytest.mark.parametrize("n,m,rho", [(4, 2, 0.9), (8, 8, 0.98), (16, 16, 0.9)])
def test_dare_limit(n, m, rho):
    rng = np.random.default_rng(5 + n)
    A, B, Q, R, x0 = rand_sys(rng, n, m, rho)
    Pinf = scipy.linalg.solve_discrete_are(A, B, Q, R)
    K, P, x, u, info = orc.solve(A, B, Q, R, x0, 400)
    assert info == 0
    np.testing.assert_allclose(P[0], Pinf, rtol=0, atol=1e-10 * np.max(np.abs(Pinf)))
    Kinf = -np.linalg.solve(R + B.T @ Pinf @ B, B.T @ Pinf @ A)
    np.testing.assert_allclose(K[0], Kinf, rtol=0, atol=1e-9)


def test_not_positive_definite_is_reported():
    n = m = 3
    A, B, Q = np.eye(n), np.eye(n), np.eye(n)
    R = np.diag([1.0, -5.0, 1.0])
    K, P, x, u, info = orc.solve(A, B, Q, R, np.ones(n), 4)
    assert info == 3 * m + 2  # first failing step is t = H-1 = 3, pivot 1 (0-based)


def test_first_only_and_batch_broadcast():
    rng = np.random.default_rng(3)
    n, m, H = 4, 3, 5
    S, Hd, T = 2, 3, 4
    sysm = [rand_sys(rng, n, m) for _ in range(Hd)]
    A = np.stack([s[0] for s in sysm]).reshape(1, Hd, 1, n, n)
    B = np.stack([s[1] for s in sysm]).reshape(1, Hd, 1, n, m)
    R = np.stack([s[3] for s in sysm]).reshape(1, Hd, 1, m, m)
    L = rng.standard_normal((S, Hd, T, n, n))
    Q = L @ np.swapaxes(L, -1, -2) / n + 0.1 * np.eye(n)
    x0 = rng.standard_normal((S, Hd, T, n))
    out = orc.solve_batch(A, B, Q, R, x0, H, nthreads=2)
    outf = orc.solve_batch(A, B, Q, R, x0, H, first_only=True, nthreads=1)
    assert out["K"].shape == (S * Hd * T, H, m, n) and outf["P"].shape == (S * Hd * T, n, n)
    i = 0
    for s in range(S):
        for h in range(Hd):
            for k in range(T):
                K1, P1, x1, u1, info = orc.solve(A[0, h, 0], B[0, h, 0], Q[s, h, k], R[0, h, 0], x0[s, h, k], H)
                assert info == 0 and out["info"][i] == 0
                assert np.array_equal(out["K"][i], K1) and np.array_equal(out["P"][i], P1)
                assert np.array_equal(out["x"][i], x1) and np.array_equal(out["u"][i], u1)
                assert np.array_equal(outf["P"][i], P1[0]) and np.array_equal(outf["u"][i], u1[0])
                i += 1
