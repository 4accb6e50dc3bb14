"""GPU parity of the time-varying solve (ttc_lqr_solve_tv) against the time-varying float64 oracle."""
import numpy as np
import pytest
import torch

from oracle import lqr_oracle as orc
from paper_2603_09221_b200 import lqr
from tests import parity_util as pu

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def tv_workload(n, m, H, batch, seed, tv=("A", "B", "Q", "R"), bf16=False):
    """Per-head A_t, B_t, R_t, per-token Q_t, Q_f, x0 (the layout of a TTC layer: dynamics and control cost belong to
    the head, state cost and initial state to the token)."""
    S, Hd, T = batch
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    rn = lambda *shape: torch.randn(shape, generator=g, device=DEV)
    th = lambda name: (H,) if name in tv else ()
    A = 0.6 * rn(1, Hd, 1, *th("A"), n, n) / np.sqrt(n) + 0.3 * torch.eye(n, device=DEV)
    B = rn(1, Hd, 1, *th("B"), n, m) / np.sqrt(n)
    M = rn(1, Hd, 1, *th("R"), m, m)
    R = M @ M.transpose(-1, -2) / m + 0.1 * torch.eye(m, device=DEV)
    R = 0.5 * (R + R.transpose(-1, -2))
    L = rn(S, Hd, T, *th("Q"), n, n)
    Q = L @ L.transpose(-1, -2) / n + 0.1 * torch.eye(n, device=DEV)
    Q = 0.5 * (Q + Q.transpose(-1, -2))
    Lf = rn(S, Hd, T, n, n)
    Qf = Lf @ Lf.transpose(-1, -2) / n + 0.05 * torch.eye(n, device=DEV)
    Qf = 0.5 * (Qf + Qf.transpose(-1, -2))
    x0 = rn(S, Hd, T, n)
    dt = torch.bfloat16 if bf16 else torch.float32
    return dict(A=A.contiguous(), B=B.contiguous(), R=R.contiguous(), Q=Q.to(dt).contiguous(), Qf=Qf.to(dt).contiguous(),
                x0=x0.to(dt).contiguous(), n=n, m=m, H=H, batch=batch, tv=tv)


def run_both(w, want=("K", "P", "x", "u", "info"), first_only=False, H=None):
    n, m, batch = w["n"], w["m"], w["batch"]
    H = w["H"] if H is None else H
    N = int(np.prod(batch))
    s = lqr.LqrSolver(n, m, w["H"], batch)
    out = lqr.alloc_outputs(n, m, H, N, DEV, first_only=first_only, want=want)
    for v in out.values():
        v.fill_(123456.0 if v.dtype == torch.float32 else -7)
    s.solve_tv(w["A"], w["B"], w["Q"], w["R"], w["Qf"], w["x0"], H, tv=w["tv"], K=out.get("K"), P=out.get("P"),
               x=out.get("x"), u=out.get("u"), info=out.get("info"), flags=lqr.TTC_OUT_FIRST_ONLY if first_only else 0)
    torch.cuda.synchronize()
    out["kernel"] = s.query(lqr.TTC_QUERY_LAST_KERNEL)
    s.close()
    f64 = lambda t: t.to(torch.float64).cpu().numpy()
    cut = lambda name: f64(w[name][..., :H, :, :] if name in w["tv"] else w[name])      # the first H time steps
    ref = orc.solve_batch_tv(cut("A"), cut("B"), cut("Q"), cut("R"), f64(w["Qf"]), f64(w["x0"]), H, batch,
                             tv=w["tv"], first_only=first_only)
    return out, ref


@pytest.mark.parametrize("n,m,H,expect", [(1, 1, 3, "riccati_cta"), (5, 3, 6, "riccati_cta"), (16, 16, 12, "riccati_warp"),
                                          (32, 32, 7, "riccati_warp"), (64, 64, 3, "riccati_cta"), (12, 16, 4, "riccati_cta")])
def test_time_varying_all_outputs(n, m, H, expect):
    w = tv_workload(n, m, H, (2, 3, 5), seed=500 + 7 * n + H)
    out, ref = run_both(w)
    assert lqr.KERNEL_NAMES[out["kernel"]] == expect
    pu.compare(out, ref, np.arange(30), 1e-4)
    for k in ("K", "P", "x", "u"):
        assert not torch.any(out[k] == 123456.0), "canary left in %s" % k


@pytest.mark.parametrize("tv", [("A",), ("Q",), ("B", "R"), ()])
@pytest.mark.parametrize("n", [8, 16])
def test_partially_time_varying_and_terminal_weight_only(n, tv):
    w = tv_workload(n, n, 9, (1, 2, 9), seed=40 + n + len(tv), tv=tv)
    out, ref = run_both(w)
    pu.compare(out, ref, np.arange(18), 1e-4)


@pytest.mark.parametrize("n", [16, 32])
def test_time_varying_first_only_bf16_and_shorter_horizon(n):
    w = tv_workload(n, n, 10, (1, 2, 7), seed=77 + n, bf16=True)
    out, ref = run_both(w, want=("P", "u", "info"), first_only=True)
    pu.compare(out, ref, np.arange(14), 2e-2, names=("P", "u"))
    out, ref = run_both(w, H=6)                      # first 6 steps of the stored 10: strides, not shapes, define the layout
    pu.compare(out, ref, np.arange(14), 2e-2)


def test_time_varying_reduces_to_time_invariant_solve_bitwise():
    w = tv_workload(16, 16, 8, (1, 2, 6), seed=5, tv=())
    s = lqr.LqrSolver(16, 16, 8, w["batch"])
    o1 = lqr.alloc_outputs(16, 16, 8, 12, DEV)
    o2 = lqr.alloc_outputs(16, 16, 8, 12, DEV)
    s.solve(w["A"], w["B"], w["Q"], w["R"], w["x0"], 8, **o1)
    s.solve_tv(w["A"], w["B"], w["Q"], w["R"], None, w["x0"], 8, tv=(), **o2)      # Q_f = Q
    torch.cuda.synchronize()
    s.close()
    for k in o1:
        assert torch.equal(o1[k], o2[k]), k


def test_scan_method_rejects_time_varying_requests():
    w = tv_workload(8, 8, 4, (1, 1, 4), seed=1)
    s = lqr.LqrSolver(8, 8, 4, w["batch"], method=lqr.TTC_SCAN)
    out = lqr.alloc_outputs(8, 8, 4, 4, DEV)
    with pytest.raises(lqr.TtcError) as ei:
        s.solve_tv(w["A"], w["B"], w["Q"], w["R"], w["Qf"], w["x0"], 4, P=out["P"])
    assert "UNSUPPORTED" in str(ei.value)
    s.close()


def test_ttc_layer_shaped_workload_full_size_on_sampled_instances():
    """The time-varying benchmark configuration (d = 16, 16 heads, horizon 32) at full size, in the launch
    configuration the benchmark times; the oracle solves a stratified sample of instances one by one."""
    from paper_2603_09221_b200 import workloads
    w = workloads.make_tv_workload("tv16", device=DEV)
    n, m, H, batch = w["n"], w["m"], w["H"], w["batch"]
    N = int(np.prod(batch))
    s = lqr.LqrSolver(n, m, H, batch)
    out = lqr.alloc_outputs(n, m, H, N, DEV, first_only=True, want=("P", "u", "info"))
    out["P"].fill_(123456.0)
    out["u"].fill_(123456.0)
    out["info"].fill_(-7)
    s.solve_tv(w["A"], w["B"], w["Q"], w["R"], w["Qf"], w["x0"], H, tv=w["tv"], P=out["P"], u=out["u"],
               info=out["info"], flags=lqr.TTC_OUT_FIRST_ONLY)
    torch.cuda.synchronize()
    assert lqr.KERNEL_NAMES[s.query(lqr.TTC_QUERY_LAST_KERNEL)] == "riccati_warp"
    assert s.query(lqr.TTC_QUERY_DEVICE_ERROR) == 0
    s.close()
    assert int(out["info"].abs().max()) == 0
    assert not torch.any(out["P"] == 123456.0) and not torch.any(out["u"] == 123456.0)
    S, Hd, T = batch
    toks = np.array([0, 1, T // 2, T - 2, T - 1])
    idx = (np.arange(S * Hd)[:, None] * T + toks[None, :]).reshape(-1)
    ref = pu.run_oracle_tv(w, idx=idx, first_only=True)
    errs = pu.compare(out, ref, idx, w["tol"], names=("P", "u"))
    print("tv16 sampled parity:", errs)
    # symmetry of P_0 holds at any size
    P = out["P"][:: 97]
    assert float((P - P.transpose(-1, -2)).abs().max() / P.abs().max()) < 1e-5


@pytest.mark.parametrize("tv,first_only,want,bf16", [(("A", "B", "Q", "R"), True, ("P", "u", "info"), False),
                                                     ((), True, ("P", "u", "info"), True),
                                                     (("Q",), False, ("P", "info"), False)])
def test_value_matrix_and_first_control_on_batches_that_fill_the_machine(tv, first_only, want, bf16):
    """n = 16, 5600 instances, P and the first control only (the shape of request the time-varying benchmark workload
    makes): several work items per CTA, 700 tokens per head leave the last work item of every head ragged.  Every
    instance against the oracle."""
    w = tv_workload(16, 16, 7, (2, 4, 700), seed=1600 + len(tv), tv=tv, bf16=bf16)
    out, ref = run_both(w, want=want, first_only=first_only)
    assert lqr.KERNEL_NAMES[out["kernel"]] == "riccati_warp"
    names = tuple(k for k in want if k != "info")
    pu.compare(out, ref, np.arange(5600), 2e-2 if bf16 else 1e-4, names=names)
    for k in names:
        assert not torch.any(out[k] == 123456.0), "canary left in %s" % k
    assert int(out["info"].abs().max()) == 0
