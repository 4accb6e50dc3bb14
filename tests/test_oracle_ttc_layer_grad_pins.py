"""Pins of the layer-gradient oracle (Thm 3.2 + the chain rule through the contextualised parameterisation):
central finite differences of the loss l = g . u_1*(coefficients) computed with the pinned FORWARD oracle
(`ttc_layer.solve`), entry by entry for every coefficient vector and along random directions for the basis matrices
(symmetric directions for Q^(k): the state cost is symmetric by definition).  A dropped term, a wrong power of the
time index, a missing factor 2 in the Gamma_Q derivative or a transposed outer product fails one of them."""
import numpy as np
import pytest

from oracle import ttc_layer as lay
from oracle import ttc_layer_grad as lg

VEC = ("s_a", "s_gamma_a", "s_gamma_b", "s_gamma_q", "s_b", "s_q", "s_qf", "r_inv", "h0")


def draw(d, r, seed):
    rng = np.random.default_rng(seed)
    sp = lambda x: np.log1p(np.exp(x))
    Qc = rng.standard_normal((r, d, d))
    return dict(s_a=0.3 * rng.standard_normal(d), s_gamma_a=sp(rng.standard_normal(d) - 2), s_gamma_b=sp(rng.standard_normal(d) - 2),
                s_gamma_q=sp(rng.standard_normal(d) - 2), s_b=rng.standard_normal(r) / np.sqrt(r), s_q=sp(rng.standard_normal(r)) / r,
                s_qf=sp(rng.standard_normal(r)) / r, r_inv=sp(rng.standard_normal(d)) + 0.5, h0=rng.standard_normal(d),
                B_basis=rng.standard_normal((r, d, d)) / np.sqrt(d), Q_basis=Qc @ np.swapaxes(Qc, 1, 2) / np.sqrt(d)), rng


def loss(p, T, g):
    out = lay.solve(p["s_a"], p["s_gamma_a"], p["s_gamma_b"], p["s_gamma_q"], p["s_b"], p["s_q"], p["s_qf"], p["r_inv"], p["h0"],
                    p["B_basis"], p["Q_basis"], T)
    assert out["info"] == 0
    return float(g @ out["u1"])


def oracle_grad(p, T, g):
    return lg.grad(p["s_a"], p["s_gamma_a"], p["s_gamma_b"], p["s_gamma_q"], p["s_b"], p["s_q"], p["s_qf"], p["r_inv"], p["h0"],
                   p["B_basis"], p["Q_basis"], T, g)


@pytest.mark.parametrize("d,r,T,seed", [(4, 3, 5, 0), (3, 2, 1, 1), (5, 4, 2, 2), (6, 2, 9, 3)])
def test_every_coefficient_gradient_matches_central_differences(d, r, T, seed):
    p, rng = draw(d, r, seed)
    g = rng.standard_normal(d)
    G = oracle_grad(p, T, g)
    assert G["info"] == 0
    fwd = lay.solve(*(p[k] for k in VEC[:8]), p["h0"], p["B_basis"], p["Q_basis"], T)
    assert np.allclose(G["u1"], fwd["u1"], rtol=1e-12, atol=1e-14)
    eps = 1e-6
    for name in VEC:
        fd = np.zeros_like(p[name])
        for i in range(p[name].shape[0]):
            hi, lo = dict(p), dict(p)
            hi[name] = p[name].copy(); hi[name][i] += eps
            lo[name] = p[name].copy(); lo[name][i] -= eps
            fd[i] = (loss(hi, T, g) - loss(lo, T, g)) / (2 * eps)
        scale = max(np.abs(fd).max(), 1e-8)
        assert np.abs(G[name] - fd).max() <= 2e-6 * scale + 1e-9, (name, G[name], fd)
    if T == 1:                                # only Q_T, A_1, B_1, R_1 exist: the running state cost has no say
        assert np.all(G["s_q"] == 0) and np.all(G["s_gamma_q"] == 0)


@pytest.mark.parametrize("d,r,T,seed", [(4, 3, 5, 10), (5, 2, 3, 11)])
def test_basis_gradients_along_random_directions(d, r, T, seed):
    p, rng = draw(d, r, seed)
    g = rng.standard_normal(d)
    G = oracle_grad(p, T, g)
    eps = 1e-6
    for name in ("B_basis", "Q_basis"):
        for _ in range(4):
            D = rng.standard_normal(p[name].shape)
            if name == "Q_basis":
                D = 0.5 * (D + np.swapaxes(D, 1, 2))
            hi, lo = dict(p), dict(p)
            hi[name] = p[name] + eps * D
            lo[name] = p[name] - eps * D
            fd = (loss(hi, T, g) - loss(lo, T, g)) / (2 * eps)
            an = float(np.sum(G[name] * D))
            assert abs(an - fd) <= 2e-6 * max(abs(fd), 1e-6), (name, an, fd)
    for k in range(r):                         # Q^(k) symmetric => its gradient is symmetric too
        assert np.allclose(G["Q_basis"][k], G["Q_basis"][k].T, rtol=0, atol=1e-13)
