"""GPU parity of ttc_lqr_grad (Thm 3.2: gradients of a loss of the first control) against the pinned gradient oracle."""
import numpy as np
import pytest
import torch

from oracle import lqr_grad as og
from paper_2603_09221_b200 import lqr
from tests import parity_util as pu
from tests.test_gpu_time_varying import tv_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
NAMES = ("dA", "dB", "dQ", "dQf", "dR", "dx0", "u0")


def shapes(n, m, H, N):
    return dict(dA=(N, H, n, n), dB=(N, H, n, m), dQ=(N, H, n, n), dQf=(N, n, n), dR=(N, H, m, m), dx0=(N, n), u0=(N, m))


def run_gpu(w, g, want=NAMES + ("info",)):
    n, m, H, batch = w["n"], w["m"], w["H"], w["batch"]
    N = int(np.prod(batch))
    s = lqr.LqrSolver(n, m, H, batch)
    out = {k: torch.full(shp, 123456.0, device=DEV) for k, shp in shapes(n, m, H, N).items() if k in want}
    if "info" in want:
        out["info"] = torch.full((N,), -7, dtype=torch.int32, device=DEV)
    s.grad(w["A"], w["B"], w["Q"], w["R"], w["Qf"], w["x0"], g, H, tv=w["tv"], **out)
    torch.cuda.synchronize()
    out["kernel"] = lqr.KERNEL_NAMES[s.query(lqr.TTC_QUERY_LAST_KERNEL)]
    out["launches"] = s.query(lqr.TTC_QUERY_LAST_LAUNCHES)
    s.close()
    return out


def run_oracle(w, g, idx=None):
    n, m, H, batch = w["n"], w["m"], w["H"], w["batch"]
    S, Hd, T = batch
    N = S * Hd * T
    f64 = lambda t: t.to(torch.float64).cpu().numpy()

    def inst(name, i, tail):
        t = w[name]
        if name in w["tv"]:
            tail = (H,) + tail
        return f64(t.expand((S, Hd, T) + tail).reshape((N,) + tail)[i])

    idx = range(N) if idx is None else idx
    refs = [og.grad(inst("A", i, (n, n)), inst("B", i, (n, m)), inst("Q", i, (n, n)), inst("R", i, (m, m)),
                    f64(w["Qf"].reshape(N, n, n)[i]), f64(w["x0"].reshape(N, n)[i]), f64(g[i]), H) for i in idx]
    return {k: np.stack([r[k] for r in refs]) for k in NAMES}


def errors(out, ref, idx=None):
    errs = {}
    for k in NAMES:
        if k in out:
            got = out[k].cpu().numpy()
            if idx is not None:
                got = got[list(idx)]
            # whole-instance norm: single time slices of a gradient can be tiny next to the others
            errs[k] = pu.block_rel_err(got.reshape(got.shape[0], -1), ref[k].reshape(got.shape[0], -1), 1, per_block=False)
    return errs


def draw_g(N, m, seed):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(seed)
    return torch.randn((N, m), generator=gen, device=DEV).contiguous()


@pytest.mark.parametrize("n,m,H", [(1, 1, 2), (5, 3, 6), (8, 8, 5), (16, 16, 12), (32, 32, 7), (12, 16, 4), (24, 20, 3), (64, 64, 3)])
def test_grad_all_outputs(n, m, H):
    batch = (2, 2, 5)
    w = tv_workload(n, m, H, batch, seed=300 + 7 * n + H)
    g = draw_g(20, m, 9)
    out = run_gpu(w, g)
    ref = run_oracle(w, g)
    errs = errors(out, ref)
    print(n, m, H, out["kernel"], errs)
    assert int(out["info"].abs().max()) == 0
    assert all(v <= 1e-4 for v in errs.values()), errs
    for k in NAMES:
        assert not torch.any(out[k] == 123456.0), "canary left in %s" % k
    assert out["kernel"] == ("riccati_warp" if n == m and n in (16, 32) else "riccati_cta")
    assert out["launches"] == 3
    assert float(out["dQ"][:, 0].abs().max()) == 0.0          # u_0 does not depend on Q_0
    for k in ("dQ", "dQf", "dR"):
        assert torch.equal(out[k], out[k].transpose(-1, -2))


@pytest.mark.parametrize("n,m,H", [(4, 4, 1), (4, 16, 2), (16, 4, 3), (16, 8, 5), (8, 16, 9), (16, 16, 1), (16, 16, 4), (32, 16, 3),
                                   (16, 32, 3), (64, 64, 1), (20, 12, 1)])
def test_grad_shapes_around_the_small_kernel(n, m, H):
    """Rectangular B_t with n, m in {4, 8, 16} (the staged kernel: different float4 counts per row for K_t, A_t, B_t),
    horizons shorter than, equal to and longer than its ring of stages, and sizes just outside it."""
    batch = (1, 3, 11)
    w = tv_workload(n, m, H, batch, seed=17 * n + 3 * m + H)
    g = draw_g(33, m, 5)
    out = run_gpu(w, g)
    ref = run_oracle(w, g)
    errs = errors(out, ref)
    assert int(out["info"].abs().max()) == 0
    assert all(v <= 1e-4 for v in errs.values()), errs
    for k in NAMES:
        assert not torch.any(out[k] == 123456.0), "canary left in %s" % k


def test_grad_per_token_dynamics():
    """A_t, B_t, R_t of every token its own (the contextualised layer's situation): no operand is shared."""
    n, m, H, batch = 16, 16, 6, (2, 2, 7)
    w = tv_workload(n, m, H, batch, seed=31)
    S, Hd, T = batch
    gen = torch.Generator(device=DEV)
    gen.manual_seed(8)
    for k in ("A", "B", "R"):
        full = w[k].expand((S, Hd, T) + w[k].shape[3:]).clone()
        if k != "R":
            full = full + 0.05 * torch.randn(full.shape, generator=gen, device=DEV)
        w[k] = full.contiguous()
    g = draw_g(28, m, 6)
    out = run_gpu(w, g)
    ref = run_oracle(w, g)
    assert out["kernel"] == "riccati_warp"                     # per-token dynamics: the warp kernel with per-instance copies
    assert all(v <= 1e-4 for v in errors(out, ref).values())


def test_grad_time_invariant_operands_and_output_subsets():
    w = tv_workload(16, 16, 9, (1, 3, 37), seed=5, tv=("Q",))                  # A, B, R constant in time, ragged chunks
    N = 111
    g = draw_g(N, 16, 4)
    ref = run_oracle(w, g)
    out = run_gpu(w, g)
    assert all(v <= 1e-4 for v in errors(out, ref).values())
    for want in (("dx0",), ("u0", "info"), ("dA", "dQf"), ("dB", "dR", "dx0")):
        o = run_gpu(w, g, want=want)
        assert o["launches"] == (2 if set(want) <= {"dx0", "u0", "info"} else 3)
        assert all(v <= 1e-4 for v in errors(o, ref).values()), want


def test_grad_is_linear_in_g_and_zero_for_zero_g():
    w = tv_workload(16, 16, 6, (1, 2, 8), seed=12)
    g = draw_g(16, 16, 1)
    a = run_gpu(w, g)
    b = run_gpu(w, 2.0 * g)
    z = run_gpu(w, torch.zeros_like(g))
    for k in ("dA", "dB", "dQ", "dQf", "dR", "dx0"):
        assert float(z[k].abs().max()) == 0.0
        torch.testing.assert_close(b[k], 2.0 * a[k], rtol=1e-5, atol=1e-6 * float(a[k].abs().max()))
    assert torch.equal(a["u0"], b["u0"]) and torch.equal(a["u0"], z["u0"])


def test_grad_bf16_state_cost_and_initial_state():
    w = tv_workload(16, 16, 8, (1, 2, 9), seed=21, bf16=True)
    g = draw_g(18, 16, 2)
    out = run_gpu(w, g)
    ref = run_oracle(w, g)                                    # the oracle sees the bf16-rounded inputs
    assert all(v <= 1e-4 for v in errors(out, ref).values())


def test_grad_failure_fills_every_output_with_nan():
    w = tv_workload(16, 16, 5, (1, 2, 9), seed=77)
    w["R"] = w["R"].clone()
    w["R"][0, 1, 0] = -50.0 * torch.eye(16, device=DEV)       # head 1: S_t loses positive definiteness
    out = run_gpu(w, draw_g(18, 16, 3))
    info = out["info"].cpu().numpy().reshape(2, 9)
    assert (info[0] == 0).all() and (info[1] != 0).all()
    for k in NAMES:
        t = out[k].reshape((2, 9) + out[k].shape[1:])
        assert torch.isnan(t[1]).all(), k
        assert torch.isfinite(t[0]).all(), k


def test_grad_full_size_sampled_instances():
    """The layer's shape (d = 16, 16 heads, horizon 32) at a few thousand tokens: sampled instances against the oracle,
    symmetry and the Q_0 property on everything."""
    batch = (2, 16, 128)
    N = 4096
    w = tv_workload(16, 16, 32, batch, seed=99)
    g = draw_g(N, 16, 8)
    out = run_gpu(w, g)
    idx = [0, 1, 127, 128, 2047, 2048, 3000, N - 1]
    ref = run_oracle(w, g, idx=idx)
    errs = errors(out, ref, idx=idx)
    assert all(v <= 1e-4 for v in errs.values()), errs
    assert int(out["info"].abs().max()) == 0
    assert float(out["dQ"][:, 0].abs().max()) == 0.0
    for k in ("dQ", "dQf", "dR"):
        assert torch.equal(out[k], out[k].transpose(-1, -2))
    for k in NAMES:
        assert torch.isfinite(out[k]).all()


@pytest.mark.parametrize("n", [8, 16, 24])
def test_null_terminal_weight_means_the_constant_state_cost(n):
    """Qf = NULL is allowed when Q is constant in time and then Q_f = Q, in all three time-varying entry points."""
    H, batch = 7, (1, 2, 6)
    w = tv_workload(n, n, H, batch, seed=70 + n, tv=("A", "B", "R"))
    N = 12
    g = draw_g(N, n, 11)
    s = lqr.LqrSolver(n, n, H, batch)
    mk = lambda *shape: torch.full(shape, 123456.0, device=DEV)
    got, exp = {}, {}
    for tag, Qf in (("null", None), ("given", w["Q"])):
        o = dict(dA=mk(N, H, n, n), dQf=mk(N, n, n), dx0=mk(N, n), u0=mk(N, n))
        s.grad(w["A"], w["B"], w["Q"], w["R"], Qf, w["x0"], g, H, tv=w["tv"], **o)
        P, u = mk(N, H + 1, n, n), mk(N, H, n)
        s.solve_tv(w["A"], w["B"], w["Q"], w["R"], Qf, w["x0"], H, tv=w["tv"], P=P, u=u)
        pv, ua = mk(N, H + 1, n), mk(N, H, n)
        r = torch.ones((1, 1, 1, n), device=DEV).expand(batch + (n,)).contiguous()
        s.solve_affine(w["A"], w["B"], w["Q"], w["R"], Qf, r, w["x0"], H, tv=w["tv"], pvec=pv, u=ua)
        torch.cuda.synchronize()
        (got if tag == "null" else exp).update(o, P=P, u=u, pv=pv, ua=ua)
    s.close()
    for k in got:
        assert not torch.any(got[k] == 123456.0), k
        assert torch.equal(got[k], exp[k]), k
    ww = dict(w, Qf=w["Q"])
    ref = run_oracle(ww, g)
    errs = errors({k: exp[k] for k in ("dA", "dQf", "dx0", "u0")}, ref)
    assert all(v <= 1e-4 for v in errs.values()), errs


def test_grad_argument_errors():
    n, m, H, batch = 8, 8, 4, (1, 1, 3)
    w = tv_workload(n, m, H, batch, seed=1)
    g = draw_g(3, m, 1)
    s = lqr.LqrSolver(n, m, H, batch)
    args = (w["A"], w["B"], w["Q"], w["R"], w["Qf"], w["x0"])
    with pytest.raises(ValueError):                                            # g of the wrong shape: caught by the binding
        s.grad(*args, g[:2], H, tv=w["tv"])
    w5 = tv_workload(n, m, H + 1, batch, seed=2)
    with pytest.raises(lqr.TtcError) as ei:                                    # horizon beyond the handle's maximum
        s.grad(w5["A"], w5["B"], w5["Q"], w5["R"], w5["Qf"], w5["x0"], g, H + 1, tv=w5["tv"])
    assert "INVALID_ARGUMENT" in str(ei.value)
    with pytest.raises(lqr.TtcError) as ei:                                    # Q_t varies in time: Qf cannot be omitted
        s.grad(w["A"], w["B"], w["Q"], w["R"], None, w["x0"], g, H, tv=w["tv"])
    assert "INVALID_ARGUMENT" in str(ei.value)
    mis = torch.empty(3 * n + 1, device=DEV)[1:].reshape(3, n)                 # 4-byte aligned only
    with pytest.raises(lqr.TtcError) as ei:
        s.grad(*args, g, H, tv=w["tv"], dx0=mis)
    assert "INVALID_ARGUMENT" in str(ei.value)
    s.close()
    s = lqr.LqrSolver(n, m, H, batch, method=lqr.TTC_SCAN)
    with pytest.raises(lqr.TtcError) as ei:
        s.grad(*args, g, H, tv=w["tv"])
    assert "UNSUPPORTED" in str(ei.value)
    s.close()
    # after the refused calls the handle still works
    out = run_gpu(w, g)
    assert all(v <= 1e-4 for v in errors(out, run_oracle(w, g)).values())
