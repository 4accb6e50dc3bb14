"""GPU parity of ttc_lqr_solve_affine (linear control cost; Prop. A.1) against the pinned affine oracle."""
import numpy as np
import pytest
import torch

from oracle import lqr_oracle as orc
from paper_2603_09221_b200 import lqr
from tests import parity_util as pu
from tests.test_gpu_time_varying import tv_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def affine_workload(n, m, H, batch, seed, tv=("A", "B", "Q", "R", "r")):
    w = tv_workload(n, m, H, batch, seed, tv=tuple(k for k in tv if k != "r"))
    S, Hd, T = batch
    g = torch.Generator(device=DEV)
    g.manual_seed(seed + 1)
    shape = (S, Hd, T) + ((H,) if "r" in tv else ()) + (m,)
    w["r"] = torch.randn(shape, generator=g, device=DEV).contiguous()
    w["tv"] = tv
    return w


def run_both(w, first_only=False, want=("K", "kff", "P", "pvec", "x", "u", "info"), with_ref=True):
    n, m, H, batch = w["n"], w["m"], w["H"], w["batch"]
    N = int(np.prod(batch))
    s = lqr.LqrSolver(n, m, H, batch)
    out = lqr.alloc_outputs(n, m, H, N, DEV, first_only=first_only, want=tuple(k for k in want if k in ("K", "P", "x", "u", "info")))
    if "kff" in want:
        out["kff"] = torch.empty((N, H, m), device=DEV)
    if "pvec" in want:
        out["pvec"] = torch.empty((N, n) if first_only else (N, H + 1, n), device=DEV)
    for v in out.values():
        v.fill_(123456.0 if v.dtype == torch.float32 else -7)
    s.solve_affine(w["A"], w["B"], w["Q"], w["R"], w["Qf"], w["r"], w["x0"], H, tv=w["tv"], K=out.get("K"), kff=out.get("kff"),
                   P=out.get("P"), pvec=out.get("pvec"), x=out.get("x"), u=out.get("u"), info=out.get("info"),
                   flags=lqr.TTC_OUT_FIRST_ONLY if first_only else 0)
    torch.cuda.synchronize()
    out["kernel"] = lqr.KERNEL_NAMES[s.query(lqr.TTC_QUERY_LAST_KERNEL)]
    s.close()
    if not with_ref:
        return out, None
    S, Hd, T = batch
    f64 = lambda t: t.to(torch.float64).cpu().numpy()

    def inst(name, i, tail):
        t = w[name]
        if name in w["tv"]:
            tail = (H,) + tail
        full = t.expand((S, Hd, T) + tail).reshape((N,) + tail)
        return f64(full[i])

    refs = [orc.solve_affine(inst("A", i, (n, n)), inst("B", i, (n, m)), inst("Q", i, (n, n)), inst("R", i, (m, m)),
                             inst("r", i, (m,)), f64(w["Qf"].reshape(N, n, n)[i]), f64(w["x0"].reshape(N, n)[i]), H)
            for i in range(N)]
    ref = {k: np.stack([r[k] for r in refs]) for k in ("K", "k", "P", "p", "x", "u")}
    return out, ref


def check(out, ref, first_only, tol=1e-4):
    errs = {}
    if "K" in out:
        errs["K"] = pu.block_rel_err(out["K"].cpu().numpy(), ref["K"], 2)
    if "kff" in out:
        errs["k"] = pu.block_rel_err(out["kff"].cpu().numpy(), ref["k"], 1, per_block=False)
    if "P" in out:
        errs["P"] = pu.block_rel_err(out["P"].cpu().numpy(), ref["P"][:, 0] if first_only else ref["P"], 2)
    if "pvec" in out:
        errs["p"] = pu.block_rel_err(out["pvec"].cpu().numpy(), ref["p"][:, 0] if first_only else ref["p"], 1, per_block=False)
    if "x" in out:
        errs["x"] = pu.block_rel_err(out["x"].cpu().numpy(), ref["x"], 1, floor=pu.XU_FLOOR)
    if "u" in out:
        errs["u"] = pu.block_rel_err(out["u"].cpu().numpy(), ref["u"][:, 0] if first_only else ref["u"], 1, floor=pu.XU_FLOOR)
    assert int(out["info"].abs().max()) == 0
    assert all(v <= tol for v in errs.values()), errs
    return errs


@pytest.mark.parametrize("n,m,H", [(1, 1, 3), (5, 3, 6), (8, 8, 5), (16, 16, 12), (32, 32, 7), (12, 16, 4), (64, 64, 3)])
def test_affine_all_outputs(n, m, H):
    w = affine_workload(n, m, H, (2, 3, 5), seed=900 + 7 * n + H)
    out, ref = run_both(w)
    errs = check(out, ref, False)
    print(n, m, H, out["kernel"], errs)
    assert out["kernel"] == ("riccati_warp" if n == m and n in (16, 32) else "riccati_cta")
    for k in ("K", "kff", "P", "pvec", "x", "u"):
        assert not torch.any(out[k] == 123456.0), "canary left in %s" % k


@pytest.mark.parametrize("n", [8, 16, 32])
def test_affine_first_only_and_constant_linear_term(n):
    w = affine_workload(n, n, 9, (1, 2, 7), seed=60 + n, tv=("A", "Q"))       # r, B, R constant in time
    out, ref = run_both(w, first_only=True, want=("P", "pvec", "u", "info"))
    check(out, ref, True)
    out2, _ = run_both(w, first_only=False, want=("x", "u", "info"))             # k_t only through the workspace
    check(out2, ref, False)


def test_zero_linear_term_matches_the_time_varying_entry_point():
    w = affine_workload(16, 16, 8, (1, 2, 6), seed=3)
    w["r"] = torch.zeros_like(w["r"])
    out, ref = run_both(w)
    check(out, ref, False)
    assert float(out["kff"].abs().max()) == 0.0 and float(out["pvec"].abs().max()) == 0.0


@pytest.mark.parametrize("n,T", [(16, 37), (32, 21)])
def test_affine_warp_kernel_ragged_chunks_and_output_subsets(n, T):
    """Several chunks of tokens per head with a ragged tail (idle segments), and the output combinations that take
    different routes through the kernel: u_0 alone (k_0 kept in a register), K with u_0 (no feed-forward buffer),
    the trajectory alone (k_t through the workspace), p_0 alone."""
    w = affine_workload(n, n, 6, (2, 2, T), seed=4242 + n)
    out, ref = run_both(w)
    assert out["kernel"] == "riccati_warp"
    check(out, ref, False)
    for first_only, want in [(True, ("u", "info")), (True, ("K", "u", "info")), (False, ("x", "info")),
                             (True, ("pvec", "info")), (True, ("kff", "u", "info"))]:
        o, _ = run_both(w, first_only=first_only, want=want)
        assert o["kernel"] == "riccati_warp"
        check(o, ref, first_only)


def test_affine_failure_fills_every_output_with_nan():
    w = affine_workload(16, 16, 5, (1, 2, 9), seed=77)
    w["R"] = w["R"].clone()
    w["R"][0, 1, 0] = -50.0 * torch.eye(16, device=DEV)           # head 1: S_t loses positive definiteness
    out, _ = run_both(w, with_ref=False)
    info = out["info"].cpu().numpy().reshape(2, 9)
    assert (info[0] == 0).all() and (info[1] != 0).all()
    for k in ("K", "kff", "P", "pvec", "x", "u"):
        t = out[k].reshape((2, 9) + out[k].shape[1:])
        assert torch.isnan(t[1]).all(), k
        assert torch.isfinite(t[0]).all(), k
