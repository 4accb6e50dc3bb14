"""Pins of the contextualised TTC-layer oracle (oracle/ttc_layer.py) against what the paper and the
mathematics fix, none of them through the oracle's own code path:

* the paper's problem statement solved by brute force (stacked dynamics, normal equations) with the
  parameter sequences rebuilt here from matrix powers of Gamma;
* the special case Gamma = I, which is a time-invariant LQR and must agree with the time-invariant oracle;
* a scalar horizon-1 closed form;
* invariances the construction implies (Q_T override, Q_0 = 0, R handed over as its inverse diagonal).
"""
import numpy as np
import pytest

from oracle import lqr_oracle as orc
from oracle import ttc_layer as lay


def draw(rng, d, r, gamma_scale=0.3):
    Bb = rng.standard_normal((r, d, d)) / np.sqrt(d)
    Qc = rng.standard_normal((r, d, d))
    Qb = Qc @ Qc.transpose(0, 2, 1) / np.sqrt(d)          # Q^(i) = Qc Qc' / sqrt(d)
    c = dict(s_a=0.3 * rng.standard_normal(d), s_ga=gamma_scale * rng.random(d), s_gb=gamma_scale * rng.random(d),
             s_gq=gamma_scale * rng.random(d), s_b=rng.standard_normal(r) / np.sqrt(r), s_q=rng.random(r) / r,
             s_qf=rng.random(r) / r, r_inv=0.5 + rng.random(d), h0=rng.standard_normal(d))
    return c, Bb, Qb


def brute_force(c, Bb, Qb, T):
    """min over u_1..u_T of sum_{t=1..T} h_t'Q_t h_t + u_t'R_t u_t, h_t = A_t h_{t-1} + B_t u_t, by stacking the
    dynamics h = Phi h0 + Psi u and solving the normal equations.  Powers of Gamma by repeated multiplication."""
    d = c["h0"].shape[0]
    Ga, Gb, Gq = (np.diag(np.exp(-c[k])) for k in ("s_ga", "s_gb", "s_gq"))
    Bbar = sum(c["s_b"][i] * Bb[i] for i in range(len(Bb)))
    Qbar = sum(c["s_q"][i] * Qb[i] for i in range(len(Qb)))
    Qfin = sum(c["s_qf"][i] * Qb[i] for i in range(len(Qb)))
    R = np.diag(1.0 / c["r_inv"])
    A, B, Q = {}, {}, {}
    pa, pb, pq = np.eye(d), np.eye(d), np.eye(d)
    for t in range(1, T + 1):
        pa, pb, pq = pa @ Ga, pb @ Gb, pq @ Gq
        A[t] = np.eye(d) + pa @ np.diag(c["s_a"])
        B[t] = Bbar @ pb
        Q[t] = pq @ Qbar @ pq
    Q[T] = Qfin
    Phi = np.zeros((T * d, d))
    Psi = np.zeros((T * d, T * d))
    for t in range(1, T + 1):
        prev_phi = np.eye(d) if t == 1 else Phi[(t - 2) * d:(t - 1) * d]
        Phi[(t - 1) * d:t * d] = A[t] @ prev_phi
        if t > 1:
            Psi[(t - 1) * d:t * d] = A[t] @ Psi[(t - 2) * d:(t - 1) * d]
        Psi[(t - 1) * d:t * d, (t - 1) * d:t * d] += B[t]
    Qs = np.zeros((T * d, T * d))
    Rs = np.zeros((T * d, T * d))
    for t in range(1, T + 1):
        Qs[(t - 1) * d:t * d, (t - 1) * d:t * d] = Q[t]
        Rs[(t - 1) * d:t * d, (t - 1) * d:t * d] = R
    Hm = Psi.T @ Qs @ Psi + Rs
    g = Psi.T @ Qs @ Phi @ c["h0"]
    u = -np.linalg.solve(Hm, g)
    h = Phi @ c["h0"] + Psi @ u
    cost = h @ Qs @ h + u @ Rs @ u
    return u.reshape(T, d), h.reshape(T, d), cost


@pytest.mark.parametrize("d,r,T", [(1, 1, 1), (2, 3, 4), (4, 2, 7), (6, 5, 5)])
def test_first_control_and_cost_match_the_stacked_problem(d, r, T):
    rng = np.random.default_rng(100 * d + T)
    c, Bb, Qb = draw(rng, d, r)
    out = lay.solve(**c, B_basis=Bb, Q_basis=Qb, T=T)
    u, h, cost = brute_force(c, Bb, Qb, T)
    assert out["info"] == 0
    np.testing.assert_allclose(out["u1"], u[0], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(out["u"], u, rtol=1e-8, atol=1e-10)
    np.testing.assert_allclose(out["h"][1:], h, rtol=1e-8, atol=1e-10)
    np.testing.assert_allclose(c["h0"] @ out["P0"] @ c["h0"], cost, rtol=1e-9)


def test_unit_gamma_is_the_time_invariant_problem():
    """s_Gamma = 0 makes every parameter constant in t; with s_Qf = s_Q the time-invariant oracle solves the same
    problem except that it also charges h_0'Q h_0: same controls, P_0 shifted by Q."""
    rng = np.random.default_rng(7)
    d, r, T = 5, 3, 6
    c, Bb, Qb = draw(rng, d, r)
    c.update(s_ga=np.zeros(d), s_gb=np.zeros(d), s_gq=np.zeros(d), s_qf=c["s_q"].copy())
    out = lay.solve(**c, B_basis=Bb, Q_basis=Qb, T=T)
    A = np.eye(d) + np.diag(c["s_a"])
    B = np.einsum("i,ijk->jk", c["s_b"], Bb)
    Q = np.einsum("i,ijk->jk", c["s_q"], Qb)
    ref = orc.solve(A, B, Q, np.diag(1.0 / c["r_inv"]), c["h0"], T)
    K, P, x, u = ref[0], ref[1], ref[2], ref[3]
    np.testing.assert_allclose(out["u"], u, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(out["P0"], P[0] - Q, rtol=1e-10, atol=1e-12)


def test_scalar_horizon_one_closed_form():
    """d = r = T = 1: u_1* = -(R + B_1^2 Q_f)^{-1} B_1 Q_f A_1 h_0 with A_1 = 1 + e^{-g_a} a, B_1 = s_b b e^{-g_b}."""
    a, ga, gb, gq, sb, sq, sqf, rinv, h0, b1, q1 = 0.4, 0.2, 0.5, 0.9, 1.3, 0.7, 0.6, 2.0, -1.5, 0.8, 1.1
    out = lay.solve([a], [ga], [gb], [gq], [sb], [sq], [sqf], [rinv], [h0], [[[b1]]], [[[q1]]], 1)
    A1 = 1.0 + np.exp(-ga) * a
    B1 = sb * b1 * np.exp(-gb)
    Qf = sqf * q1
    R = 1.0 / rinv
    u1 = -(B1 * Qf * A1 * h0) / (R + B1 * B1 * Qf)
    np.testing.assert_allclose(out["u1"], [u1], rtol=1e-13)
    P0 = A1 * Qf * A1 - (A1 * Qf * B1) ** 2 / (R + B1 * B1 * Qf)
    np.testing.assert_allclose(out["P0"], [[P0]], rtol=1e-13)


def test_terminal_override_and_zero_initial_weight():
    rng = np.random.default_rng(11)
    d, r = 3, 4
    c, Bb, Qb = draw(rng, d, r)
    # T = 1: the only state weight is Q_T = sum s_Qf Q^(i); s_Q and s_GammaQ must not matter
    base = lay.solve(**c, B_basis=Bb, Q_basis=Qb, T=1)
    c2 = dict(c, s_q=rng.random(r), s_gq=rng.random(d))
    other = lay.solve(**c2, B_basis=Bb, Q_basis=Qb, T=1)
    np.testing.assert_allclose(base["u1"], other["u1"], rtol=1e-13)
    np.testing.assert_allclose(base["P0"], other["P0"], rtol=1e-13)
    # T = 2: Q_1 = Gamma_Q Qbar Gamma_Q does matter
    b2 = lay.solve(**c, B_basis=Bb, Q_basis=Qb, T=2)
    o2 = lay.solve(**c2, B_basis=Bb, Q_basis=Qb, T=2)
    assert np.abs(b2["u1"] - o2["u1"]).max() > 1e-6
    # Q_0 = 0: P_0 = A_1' (...) A_1 vanishes on the kernel of A_1.  Make A_1 singular in coordinate 0.
    c3 = dict(c, s_a=c["s_a"].copy())
    c3["s_a"][0] = -np.exp(c["s_ga"][0])               # 1 + e^{-g} a = 0
    o3 = lay.solve(**c3, B_basis=Bb, Q_basis=Qb, T=3)
    e0 = np.zeros(d); e0[0] = 1.0
    assert abs(e0 @ o3["P0"] @ e0) < 1e-12


def test_synthesis_structure():
    rng = np.random.default_rng(3)
    d, r, T = 4, 3, 9
    c, Bb, Qb = draw(rng, d, r, gamma_scale=1.0)
    A, B, Q, R = lay.synthesize(*(c[k] for k in ("s_a", "s_ga", "s_gb", "s_gq", "s_b", "s_q", "s_qf", "r_inv")), Bb, Qb, T)
    assert np.all(Q[0] == 0.0)
    Bbar = np.einsum("i,ijk->jk", c["s_b"], Bb)
    for t in range(1, T + 1):
        assert np.allclose(A[t], np.diag(np.diag(A[t])))                       # diagonal A_t
        assert np.allclose(R[t] @ np.diag(c["r_inv"]), np.eye(d))              # R_t^{-1} = diag(r_inv)
        assert np.allclose(B[t], Bbar * np.exp(-c["s_gb"])[None, :] ** t)      # columns of Bbar discounted t times
        assert np.linalg.eigvalsh(0.5 * (Q[t] + Q[t].T)).min() > -1e-12        # PSD
    # discounting: |A_t - I| and |Q_t| decay monotonically for t < T
    dev = [np.abs(A[t] - np.eye(d)).max() for t in range(1, T + 1)]
    assert all(x >= y for x, y in zip(dev, dev[1:]))
    qn = [np.abs(Q[t]).max() for t in range(1, T)]
    assert all(x >= y for x, y in zip(qn, qn[1:]))
    np.testing.assert_allclose(Q[T], np.einsum("i,ijk->jk", c["s_qf"], Qb))


def test_batch_matches_single():
    rng = np.random.default_rng(5)
    d, r, T, N = 4, 3, 6, 7
    _, Bb, Qb = draw(rng, d, r)
    cs = [draw(rng, d, r)[0] for _ in range(N)]
    stack = {k: np.stack([c[k] for c in cs]) for k in cs[0]}
    out = lay.solve_batch(**stack, B_basis=Bb, Q_basis=Qb, T=T)
    for i, c in enumerate(cs):
        one = lay.solve(**c, B_basis=Bb, Q_basis=Qb, T=T)
        np.testing.assert_array_equal(out["u1"][i], one["u1"])
        np.testing.assert_array_equal(out["P0"][i], one["P0"])


def test_first_control_matches_the_symplectic_iteration_theorem():
    """Thm 3.3: u_1* = -R_1^{-1} B_1' A_1^{-T} Y1^{-1} Y2 h_0 with [Y1 Y2] = [I Q_T] Sigma_T ... Sigma_1, evaluated by
    the oracle's restatement of Alg. 3 (a different algorithm from the backward recursion the layer oracle uses).
    Short horizons only: the product is a shooting method and loses accuracy as T grows (printed, not asserted)."""
    from oracle import symplectic as sym
    rng = np.random.default_rng(21)
    d, r = 6, 4
    worst = {}
    for T in (1, 3, 6, 24):
        errs = []
        for _ in range(8):
            c, Bb, Qb = draw(rng, d, r)
            A, B, Q, R = lay.synthesize(*(c[k] for k in ("s_a", "s_ga", "s_gb", "s_gq", "s_b", "s_q", "s_qf", "r_inv")), Bb, Qb, T)
            Y1, Y2, lam0, u1 = sym.reverse_symplectic(A[1:], B[1:], Q, R[1:], c["h0"])
            P0 = np.linalg.solve(Y1, Y2)
            out = lay.solve(**c, B_basis=Bb, Q_basis=Qb, T=T)
            errs.append(max(np.abs(u1 - out["u1"]).max() / np.abs(out["u1"]).max(),
                            np.abs(P0 - out["P0"]).max() / np.abs(out["P0"]).max()))
        worst[T] = max(errs)
    print("symplectic iteration vs backward recursion, max relative difference by horizon:", worst)
    assert worst[1] < 1e-10 and worst[3] < 1e-9 and worst[6] < 1e-7
