"""Pins of the gradient oracle (Thm 3.2), none of them through its own formulas: central finite differences of
the pinned forward solve (directional and entry by entry), the dense KKT system of the theorem's proof solved as one
linear system for both the primal and the dual solution (states, controls and co-states), and a scalar closed form."""
import numpy as np
import pytest

from oracle import lqr_grad as og
from oracle import lqr_oracle as orc


def draw(rng, n, m, H):
    A = 0.6 * rng.standard_normal((H, n, n)) / np.sqrt(n) + 0.3 * np.eye(n)
    B = rng.standard_normal((H, n, m)) / np.sqrt(n)
    M = rng.standard_normal((H, m, m)); R = M @ M.transpose(0, 2, 1) / m + 0.2 * np.eye(m)
    L = rng.standard_normal((H, n, n)); Q = L @ L.transpose(0, 2, 1) / n + 0.1 * np.eye(n)
    Lf = rng.standard_normal((n, n)); Qf = Lf @ Lf.T / n + 0.1 * np.eye(n)
    return dict(A=A, B=B, Q=Q, R=R, Qf=Qf, x0=rng.standard_normal(n))


def loss(th, g, H):
    K, P, x, u, info = orc.solve_tv(th["A"], th["B"], th["Q"], th["R"], th["Qf"], th["x0"], H)
    assert info == 0
    return float(g @ u[0])


def sym(D):
    return 0.5 * (D + np.swapaxes(D, -1, -2))


GRAD_OF = dict(A="dA", B="dB", Q="dQ", R="dR", Qf="dQf", x0="dx0")


@pytest.mark.parametrize("n,m,H", [(1, 1, 1), (2, 1, 3), (3, 2, 4), (4, 4, 6), (6, 3, 5)])
def test_directional_derivatives_match_central_differences(n, m, H):
    rng = np.random.default_rng(100 * n + 10 * m + H)
    th = draw(rng, n, m, H)
    g = rng.standard_normal(m)
    out = og.grad(th["A"], th["B"], th["Q"], th["R"], th["Qf"], th["x0"], g, H)
    assert out["info"] == 0
    eps = 1e-5
    for name in ("A", "B", "Q", "R", "Qf", "x0"):
        for trial in range(3):
            D = rng.standard_normal(th[name].shape)
            if name in ("Q", "R", "Qf"):
                D = sym(D)
            if trial == 2 and name in ("A", "B", "Q", "R"):
                D[:] = D[0]                                  # the same perturbation at every t: a time-invariant matrix
            up = dict(th); dn = dict(th)
            up[name] = th[name] + eps * D
            dn[name] = th[name] - eps * D
            fd = (loss(up, g, H) - loss(dn, g, H)) / (2 * eps)
            an = float(np.sum(out[GRAD_OF[name]] * D))
            assert abs(fd - an) <= 2e-7 * (1.0 + abs(an)), (name, trial, fd, an)


def test_every_entry_on_a_tiny_problem():
    n, m, H = 2, 2, 3
    rng = np.random.default_rng(5)
    th = draw(rng, n, m, H)
    g = rng.standard_normal(m)
    out = og.grad(th["A"], th["B"], th["Q"], th["R"], th["Qf"], th["x0"], g, H)
    eps = 1e-5
    for name in ("A", "B", "Q", "R", "Qf", "x0"):
        G = out[GRAD_OF[name]]
        for idx in np.ndindex(th[name].shape):
            D = np.zeros(th[name].shape)
            D[idx] = 1.0
            if name in ("Q", "R", "Qf"):
                D = sym(D)
            up = dict(th); dn = dict(th)
            up[name] = th[name] + eps * D
            dn[name] = th[name] - eps * D
            fd = (loss(up, g, H) - loss(dn, g, H)) / (2 * eps)
            assert abs(fd - G[idx]) <= 2e-7 * (1.0 + abs(G[idx])), (name, idx, fd, G[idx])
    assert np.abs(out["dQ"][0]).max() == 0.0                 # the first control does not depend on Q_0


def kkt_matrix(th, H):
    """The linear system of the proof of Thm 3.2: variables z = [x_0..x_H, u_0..u_{H-1}], multipliers xi_0..xi_H of
    the constraints  -x_0 = -x_init,  A_t x_t - x_{t+1} + B_t u_t = 0."""
    A, B, Q, R, Qf = th["A"], th["B"], th["Q"], th["R"], th["Qf"]
    n, m = B.shape[-2:]
    nz = (H + 1) * n + H * m
    C = np.zeros((nz, nz)); F = np.zeros(((H + 1) * n, nz))
    xs = lambda t: slice(t * n, (t + 1) * n)
    us = lambda t: slice((H + 1) * n + t * m, (H + 1) * n + (t + 1) * m)
    for t in range(H):
        C[xs(t), xs(t)] = Q[t]
        C[us(t), us(t)] = R[t]
    C[xs(H), xs(H)] = Qf
    F[xs(0), xs(0)] = -np.eye(n)
    for t in range(H):
        F[xs(t + 1), xs(t)] = A[t]
        F[xs(t + 1), xs(t + 1)] = -np.eye(n)
        F[xs(t + 1), us(t)] = B[t]
    Kmat = np.block([[C, F.T], [F, np.zeros((F.shape[0],) * 2)]])
    return Kmat, nz, xs, us


@pytest.mark.parametrize("n,m,H", [(2, 1, 3), (3, 3, 5), (5, 2, 4)])
def test_primal_and_dual_kkt_solutions_against_one_dense_solve(n, m, H):
    rng = np.random.default_rng(7 * n + H)
    th = draw(rng, n, m, H)
    g = rng.standard_normal(m)
    out = og.grad(th["A"], th["B"], th["Q"], th["R"], th["Qf"], th["x0"], g, H)
    Kmat, nz, xs, us = kkt_matrix(th, H)
    rhs = np.zeros(Kmat.shape[0]); rhs[nz:nz + n] = -th["x0"]
    sol = np.linalg.solve(Kmat, rhs)
    rhs_d = np.zeros(Kmat.shape[0]); rhs_d[us(0)] = -g         # stationarity of the dual: C z + F'xi + [0; g at u_0] = 0
    sol_d = np.linalg.solve(Kmat, rhs_d)
    for s, (xk, uk, lk) in ((sol, ("x", "u", "lam")), (sol_d, ("xd", "ud", "lamd"))):
        np.testing.assert_allclose(s[:(H + 1) * n].reshape(H + 1, n), out[xk], rtol=0, atol=1e-10)
        np.testing.assert_allclose(s[(H + 1) * n:nz].reshape(H, m), out[uk], rtol=0, atol=1e-10)
        np.testing.assert_allclose(s[nz:].reshape(H + 1, n), out[lk], rtol=0, atol=1e-10)


def test_scalar_one_step_closed_form():
    a, b, q0, r, qf, x0, g = 0.7, -1.3, 0.4, 0.9, 1.6, 2.5, -0.8
    out = og.grad(np.array([[a]]), np.array([[b]]), np.array([[q0]]), np.array([[r]]), np.array([[qf]]), np.array([x0]),
                  np.array([g]), 1)
    S = r + b * b * qf
    assert out["u0"][0] == pytest.approx(-a * b * qf * x0 / S, rel=1e-13)
    assert out["dA"][0, 0, 0] == pytest.approx(g * (-b * qf * x0 / S), rel=1e-12)
    assert out["dB"][0, 0, 0] == pytest.approx(g * (-a * qf * x0 * (r - b * b * qf) / S ** 2), rel=1e-12)
    assert out["dQf"][0, 0] == pytest.approx(g * (-a * b * x0 * r / S ** 2), rel=1e-12)
    assert out["dR"][0, 0, 0] == pytest.approx(g * (a * b * qf * x0 / S ** 2), rel=1e-12)
    assert out["dx0"][0] == pytest.approx(g * (-a * b * qf / S), rel=1e-12)
    assert out["dQ"][0, 0, 0] == 0.0


def test_planted_mistakes_are_caught():
    """The finite-difference pin separates the theorem's formulas from their plausible corruptions."""
    n, m, H = 3, 2, 4
    rng = np.random.default_rng(11)
    th = draw(rng, n, m, H)
    g = rng.standard_normal(m)
    out = og.grad(th["A"], th["B"], th["Q"], th["R"], th["Qf"], th["x0"], g, H)
    x, u, lam, xd, ud, lamd = (out[k] for k in ("x", "u", "lam", "xd", "ud", "lamd"))
    wrong = dict(
        shifted_costate=np.stack([np.outer(lam[t], xd[t]) + np.outer(lamd[t], x[t]) for t in range(H)]),
        dropped_term=np.stack([np.outer(lamd[t + 1], x[t]) for t in range(H)]),
        transposed=np.stack([np.outer(xd[t], lam[t + 1]) + np.outer(x[t], lamd[t + 1]) for t in range(H)]),
        doubled_costate=np.stack([np.outer(2 * lam[t + 1], xd[t]) + np.outer(lamd[t + 1], x[t]) for t in range(H)]))
    eps = 1e-5
    D = rng.standard_normal(th["A"].shape)
    up = dict(th); dn = dict(th)
    up["A"] = th["A"] + eps * D; dn["A"] = th["A"] - eps * D
    fd = (loss(up, g, H) - loss(dn, g, H)) / (2 * eps)
    assert abs(fd - np.sum(out["dA"] * D)) <= 2e-7 * (1 + abs(fd))
    for name, G in wrong.items():
        assert abs(fd - np.sum(G * D)) > 1e-3 * (1 + abs(fd)), name
