"""Pins of the affine-cost oracle (lqr_oracle_solve_affine: Definition A.1 with r_t, Prop. A.1), none of them
through its own recursion: the stacked quadratic program solved directly, the r = 0 reduction to the pinned
time-varying routine, a scalar closed form, and the first-order optimality of the returned trajectory."""
import numpy as np
import pytest

from oracle import lqr_oracle as orc


def draw(rng, n, m, H):
    A = 0.6 * rng.standard_normal((H, n, n)) / np.sqrt(n) + 0.3 * np.eye(n)
    B = rng.standard_normal((H, n, m)) / np.sqrt(n)
    M = rng.standard_normal((H, m, m)); R = M @ M.transpose(0, 2, 1) / m + 0.2 * np.eye(m)
    L = rng.standard_normal((H, n, n)); Q = L @ L.transpose(0, 2, 1) / n + 0.1 * np.eye(n)
    Lf = rng.standard_normal((n, n)); Qf = Lf @ Lf.T / n + 0.1 * np.eye(n)
    return A, B, Q, R, rng.standard_normal((H, m)), Qf, rng.standard_normal(n)


def stacked(A, B, Q, R, r, Qf, x0):
    """min over u of sum_t 1/2 (x_t'Q_t x_t + u_t'R_t u_t) + r_t'u_t + 1/2 x_H'Qf x_H with x = Phi x0 + Psi u."""
    H, n, m = B.shape
    Phi = np.zeros(((H + 1) * n, n)); Psi = np.zeros(((H + 1) * n, H * m))
    Phi[:n] = np.eye(n)
    for t in range(H):
        Phi[(t + 1) * n:(t + 2) * n] = A[t] @ Phi[t * n:(t + 1) * n]
        Psi[(t + 1) * n:(t + 2) * n] = A[t] @ Psi[t * n:(t + 1) * n]
        Psi[(t + 1) * n:(t + 2) * n, t * m:(t + 1) * m] += B[t]
    Qs = np.zeros(((H + 1) * n,) * 2); Rs = np.zeros((H * m,) * 2)
    for t in range(H):
        Qs[t * n:(t + 1) * n, t * n:(t + 1) * n] = Q[t]
        Rs[t * m:(t + 1) * m, t * m:(t + 1) * m] = R[t]
    Qs[H * n:, H * n:] = Qf
    Hm = Psi.T @ Qs @ Psi + Rs
    g = Psi.T @ Qs @ Phi @ x0 + r.reshape(-1)
    u = -np.linalg.solve(Hm, g)
    x = Phi @ x0 + Psi @ u
    cost = 0.5 * (x @ Qs @ x + u @ Rs @ u) + r.reshape(-1) @ u
    return u.reshape(H, m), x.reshape(H + 1, n), cost


@pytest.mark.parametrize("n,m,H", [(1, 1, 1), (2, 1, 3), (3, 2, 5), (5, 4, 7), (4, 6, 4)])
def test_trajectory_and_cost_match_the_stacked_program(n, m, H):
    rng = np.random.default_rng(10 * n + m + H)
    A, B, Q, R, r, Qf, x0 = draw(rng, n, m, H)
    out = orc.solve_affine(A, B, Q, R, r, Qf, x0, H)
    u, x, cost = stacked(A, B, Q, R, r, Qf, x0)
    assert out["info"] == 0
    np.testing.assert_allclose(out["u"], u, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(out["x"], x, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(out["u"][0], out["K"][0] @ x0 + out["k"][0], rtol=1e-12, atol=1e-13)
    # V_0(x) = 1/2 x'P_0 x + p_0'x + c_0: differences of the optimal cost between initial states pin P_0 and p_0
    d = rng.standard_normal(n)
    c_plus = stacked(A, B, Q, R, r, Qf, x0 + d)[2]
    c_minus = stacked(A, B, Q, R, r, Qf, x0 - d)[2]
    np.testing.assert_allclose(c_plus - c_minus, 2 * (x0 @ out["P"][0] @ d + out["p"][0] @ d), rtol=1e-8, atol=1e-10)
    np.testing.assert_allclose(c_plus + c_minus - 2 * cost, d @ out["P"][0] @ d, rtol=1e-8, atol=1e-10)


def test_zero_linear_term_is_the_time_varying_routine():
    rng = np.random.default_rng(4)
    n, m, H = 4, 3, 6
    A, B, Q, R, r, Qf, x0 = draw(rng, n, m, H)
    out = orc.solve_affine(A, B, Q, R, np.zeros((H, m)), Qf, x0, H)
    K, P, x, u, info = orc.solve_tv(A, B, Q, R, Qf, x0, H)
    assert np.array_equal(out["K"], K) and np.array_equal(out["P"], P)
    np.testing.assert_allclose(out["x"], x, rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(out["u"], u, rtol=1e-14, atol=1e-15)
    assert np.all(out["k"] == 0) and np.all(out["p"] == 0)


def test_scalar_horizon_one_closed_form():
    a, b, q, rr, r, qf, x0 = 0.7, 1.3, 0.4, 0.5, -0.8, 1.1, 2.0
    out = orc.solve_affine([[a]], [[b]], [[q]], [[rr]], [r], [[qf]], [x0], 1)
    S = rr + b * b * qf
    u0 = -(b * qf * a * x0 + r) / S                  # minimiser of 1/2 rr u^2 + r u + 1/2 qf (a x0 + b u)^2
    np.testing.assert_allclose(out["u"], [[u0]], rtol=1e-14)
    np.testing.assert_allclose(out["k"], [[-r / S]], rtol=1e-14)
    np.testing.assert_allclose(out["p"][0], [-a * qf * b * r / S], rtol=1e-14)


def test_first_order_optimality_with_costates():
    """lambda_t = Q_t x_t + A_t' lambda_{t+1} (lambda_H = Qf x_H) and R_t u_t + r_t + B_t' lambda_{t+1} = 0."""
    rng = np.random.default_rng(8)
    n, m, H = 5, 3, 6
    A, B, Q, R, r, Qf, x0 = draw(rng, n, m, H)
    out = orc.solve_affine(A, B, Q, R, r, Qf, x0, H)
    lam = Qf @ out["x"][H]
    for t in range(H - 1, -1, -1):
        res = R[t] @ out["u"][t] + r[t] + B[t].T @ lam
        assert np.abs(res).max() < 1e-10
        # lambda_{t+1} = P_{t+1} x_{t+1} + p_{t+1}
        np.testing.assert_allclose(lam, out["P"][t + 1] @ out["x"][t + 1] + out["p"][t + 1], rtol=1e-9, atol=1e-11)
        lam = Q[t] @ out["x"][t] + A[t].T @ lam
