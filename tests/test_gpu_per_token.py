"""A, B, R that belong to the token instead of the head (the contextualised layer's situation, given as dense matrices):
the fp32 warp kernel keeps a copy per instance.  Parity of every entry point that can receive such operands."""
import numpy as np
import pytest
import torch

from oracle import lqr_oracle as orc
from paper_2603_09221_b200 import lqr
from tests import parity_util as pu
from tests.test_gpu_time_varying import tv_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def per_token(w, seed, keys=("A", "B", "R")):
    S, Hd, T = w["batch"]
    gen = torch.Generator(device=DEV)
    gen.manual_seed(seed)
    w = dict(w)
    for k in keys:
        full = w[k].expand((S, Hd, T) + w[k].shape[3:]).clone()
        if k != "R":
            full = full + 0.05 * torch.randn(full.shape, generator=gen, device=DEV)
        else:
            full = full * (1.0 + 0.2 * torch.rand((S, Hd, T) + (1,) * (full.dim() - 3), generator=gen, device=DEV))
        w[k] = full.contiguous()
    return w


def oracle_tv(w, H, first_only):
    n, m, batch = w["n"], w["m"], w["batch"]
    f64 = lambda t: t.to(torch.float64).cpu().numpy()
    return orc.solve_batch_tv(f64(w["A"]), f64(w["B"]), f64(w["Q"]), f64(w["R"]), f64(w["Qf"]), f64(w["x0"]), H, batch,
                              tv=w["tv"], first_only=first_only)


@pytest.mark.parametrize("n,H,T,tv", [(16, 9, 37, ("A", "B", "Q", "R")), (32, 5, 13, ("A", "B", "Q", "R")),
                                      (16, 6, 8, ("Q",)), (32, 4, 5, ("A", "Q"))])
def test_per_token_time_varying_solve(n, H, T, tv):
    batch = (2, 2, T)
    w = per_token(tv_workload(n, n, H, batch, seed=40 + n + H, tv=tv), seed=5)
    N = int(np.prod(batch))
    for first_only in (False, True):
        want = ("P", "u", "info") if first_only else ("K", "P", "x", "u", "info")
        s = lqr.LqrSolver(n, n, H, batch)
        out = lqr.alloc_outputs(n, n, H, N, DEV, first_only=first_only, want=want)
        for v in out.values():
            v.fill_(123456.0 if v.dtype == torch.float32 else -7)
        s.solve_tv(w["A"], w["B"], w["Q"], w["R"], w["Qf"], w["x0"], H, tv=tv, K=out.get("K"), P=out.get("P"), x=out.get("x"),
                   u=out.get("u"), info=out.get("info"), flags=lqr.TTC_OUT_FIRST_ONLY if first_only else 0)
        torch.cuda.synchronize()
        assert lqr.KERNEL_NAMES[s.query(lqr.TTC_QUERY_LAST_KERNEL)] == "riccati_warp"
        s.close()
        ref = oracle_tv(w, H, first_only)
        names = tuple(k for k in want if k != "info")
        errs = pu.compare(out, ref, np.arange(N), 1e-4, names=names)
        for k in names:
            assert not torch.any(out[k] == 123456.0), k
        print(n, H, tv, first_only, errs)


@pytest.mark.parametrize("n", [16, 32])
def test_per_token_time_invariant_solve(n):
    """ttc_lqr_solve with a system per instance (no time axis at all)."""
    H, batch = 10, (1, 3, 11)
    w = per_token(tv_workload(n, n, H, batch, seed=9 + n, tv=()), seed=2)
    N = 33
    s = lqr.LqrSolver(n, n, H, batch)
    out = lqr.alloc_outputs(n, n, H, N, DEV, first_only=False, want=("K", "P", "x", "u", "info"))
    s.solve(w["A"], w["B"], w["Q"], w["R"], w["x0"], H, K=out["K"], P=out["P"], x=out["x"], u=out["u"], info=out["info"])
    torch.cuda.synchronize()
    assert lqr.KERNEL_NAMES[s.query(lqr.TTC_QUERY_LAST_KERNEL)] == "riccati_warp"
    s.close()
    f64 = lambda t: t.to(torch.float64).cpu().numpy()
    ref = orc.solve_batch(f64(w["A"]), f64(w["B"]), f64(w["Q"]), f64(w["R"]), f64(w["x0"]), H, batch=batch)
    pu.compare(out, ref, np.arange(N), 1e-4)


def test_per_token_linear_cost():
    from tests.test_gpu_affine import affine_workload, run_both, check
    w = per_token(affine_workload(16, 16, 7, (1, 2, 9), seed=77), seed=3)
    out, ref = run_both(w)
    assert out["kernel"] == "riccati_warp"
    check(out, ref, False)
    out, ref = run_both(w, first_only=True, want=("P", "pvec", "u", "info"))
    check(out, ref, True)


def test_mixed_sharing_goes_to_the_generic_kernel():
    """A per token but B, R per head: neither layout of the warp kernel applies."""
    H, batch = 5, (1, 2, 6)
    w = per_token(tv_workload(16, 16, H, batch, seed=4), seed=1, keys=("A",))
    s = lqr.LqrSolver(16, 16, H, batch)
    out = lqr.alloc_outputs(16, 16, H, 12, DEV, first_only=False, want=("K", "P", "x", "u", "info"))
    s.solve_tv(w["A"], w["B"], w["Q"], w["R"], w["Qf"], w["x0"], H, tv=w["tv"], K=out["K"], P=out["P"], x=out["x"], u=out["u"],
               info=out["info"])
    torch.cuda.synchronize()
    assert lqr.KERNEL_NAMES[s.query(lqr.TTC_QUERY_LAST_KERNEL)] == "riccati_cta"
    s.close()
    pu.compare(out, oracle_tv(w, H, False), np.arange(12), 1e-4)
