"""Compact inputs and outputs: bfloat16 outputs (TTC_OUT_BF16) and the state cost handed over as
Q = scale * U U' + diag(d) (ttc_lqr_solve_lowrank_q).  Both go through the same kernels as the plain call, so the
bfloat16 outputs must be the float32 outputs rounded to nearest even, bit for bit, and the factored operand must give
what the dense float64 oracle gives on the Q it describes."""
import numpy as np
import pytest
import torch

from oracle import lqr_oracle as orc
from paper_2603_09221_b200 import lqr, workloads
from tests import parity_util as pu
from tests.test_gpu_parity import small_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def solve(w, H, first_only, want, dtype, method=lqr.TTC_AUTO):
    n, m = w["n"], w["m"]
    N = int(np.prod(w["batch"]))
    s = lqr.LqrSolver(n, m, H, w["batch"], method=method)
    out = lqr.alloc_outputs(n, m, H, N, DEV, first_only=first_only, want=want, dtype=dtype)
    for k, v in out.items():
        v.fill_(-7 if k == "info" else 12345.0)
    flags = (lqr.TTC_OUT_FIRST_ONLY if first_only else 0) | (lqr.TTC_OUT_BF16 if dtype == torch.bfloat16 else 0)
    try:
        s.solve(w["A"], w["B"], w["Q"], w["R"], w["x0"], H, K=out.get("K"), P=out.get("P"), x=out.get("x"), u=out.get("u"),
                info=out.get("info"), flags=flags)
        torch.cuda.synchronize()
        out["kernel"] = lqr.KERNEL_NAMES[s.query(lqr.TTC_QUERY_LAST_KERNEL)]
    finally:
        s.close()
    return out


@pytest.mark.parametrize("n,H,batch,bf16_in", [(16, 9, (2, 3, 11), False), (32, 6, (1, 2, 9), False), (64, 5, (1, 2, 13), True)])
@pytest.mark.parametrize("first_only", [False, True])
def test_bfloat16_outputs_are_the_rounded_float32_outputs(n, H, batch, bf16_in, first_only):
    w = small_workload(n, n, H, batch, seed=300 + n, bf16=bf16_in)
    N = int(np.prod(batch))
    want = ("P", "u", "info") if first_only else ("K", "P", "x", "u", "info")
    full = solve(w, H, first_only, want, torch.float32)
    half = solve(w, H, first_only, want, torch.bfloat16)
    assert half["kernel"] == full["kernel"] and half["kernel"] in ("riccati_warp", "riccati_umma")
    for k in want[:-1]:
        assert half[k].dtype == torch.bfloat16 and not torch.any(half[k] == 12345.0), k
        assert torch.equal(half[k], full[k].to(torch.bfloat16)), k                 # round to nearest even, bit for bit
    assert torch.equal(half["info"], full["info"]) and int(full["info"].abs().max()) == 0
    ref = pu.run_oracle(w, first_only=first_only, H=H)
    widened = {k: half[k].float() for k in want[:-1]}
    widened["info"] = half["info"]
    pu.compare(widened, ref, np.arange(N), w["tol"] + 2.0 ** -8, names=want[:-1])   # + half an ulp of bfloat16


def test_bfloat16_outputs_of_a_failed_instance_are_nan_and_unsupported_requests_are_refused():
    w = small_workload(16, 16, 5, (1, 1, 6), seed=12)
    w["Q"] = w["Q"].clone()
    w["Q"][0, 0, 2] = -torch.eye(16, device=DEV) * 50.0          # indefinite state cost: R + B'PB loses definiteness
    out = solve(w, 5, False, ("K", "P", "x", "u", "info"), torch.bfloat16)
    assert int(out["info"][2]) > 0 and int(out["info"].abs().sum()) == int(out["info"][2])
    for k in ("K", "P", "x", "u"):
        assert bool(torch.isnan(out[k][2].float()).all()) and not bool(torch.isnan(out[k][[0, 1, 3, 4, 5]].float()).any())
    for kw in (dict(n=8, method=lqr.TTC_AUTO), dict(n=16, method=lqr.TTC_SCAN)):
        w2 = small_workload(kw["n"], kw["n"], 4, (1, 1, 5), seed=3)
        with pytest.raises(lqr.TtcError) as ei:
            solve(w2, 4, False, ("K", "P", "x", "u", "info"), torch.bfloat16, method=kw["method"])
        assert "UNSUPPORTED" in str(ei.value)


@pytest.mark.parametrize("n,rank,H,batch,bf16", [(64, 8, 6, (1, 2, 21), True), (16, 4, 7, (2, 2, 9), False), (32, 32, 4, (1, 1, 7), False)])
def test_low_rank_plus_diagonal_state_cost(n, rank, H, batch, bf16):
    w = small_workload(n, n, H, batch, seed=640 + n + rank, bf16=bf16)
    N = int(np.prod(batch))
    g = torch.Generator(device=DEV)
    g.manual_seed(5 + n)
    dt = torch.bfloat16 if bf16 else torch.float32
    U = torch.randn(batch + (n, rank), generator=g, device=DEV).to(dt)
    d = (0.05 + 0.15 * torch.rand(batch + (n,), generator=g, device=DEV)).to(dt)
    scale = 1.0 / rank
    s = lqr.LqrSolver(n, n, H, batch)
    out = lqr.alloc_outputs(n, n, H, N, DEV)
    s.solve_lowrank_q(w["A"], w["B"], U, d, scale, w["R"], w["x0"], H, **out)
    torch.cuda.synchronize()
    kernel = lqr.KERNEL_NAMES[s.query(lqr.TTC_QUERY_LAST_KERNEL)]
    s.close()
    assert kernel == ("riccati_umma" if n == 64 else "riccati_warp")
    # the oracle gets the dense Q the factors describe, formed in float64 from the very numbers the GPU was given
    U64, d64 = U.double().cpu().numpy(), d.double().cpu().numpy()
    Q64 = scale * U64 @ np.swapaxes(U64, -1, -2) + d64[..., None] * np.eye(n)
    f64 = lambda t: t.double().cpu().numpy()
    ref = orc.solve_batch(f64(w["A"]), f64(w["B"]), Q64, f64(w["R"]), f64(w["x0"]), H, batch=batch)
    pu.compare(out, ref, np.arange(N), w["tol"])


@pytest.mark.parametrize("n,H,batch,bf16_in,first_only", [(32, 6, (1, 2, 9), False, True), (64, 4, (1, 2, 512), True, False)])
def test_host_buffer_entry_point_with_bfloat16_outputs(n, H, batch, bf16_in, first_only):
    """TTC_OUT_BF16 through ttc_lqr_solve_host (one slice, and the sliced pipeline at n = 64): the host arrays hold
    bfloat16 and equal the device entry point's bfloat16 outputs bit for bit."""
    w = small_workload(n, n, H, batch, seed=400 + n, bf16=bf16_in)
    N = int(np.prod(batch))
    want = ("P", "u", "info") if first_only else ("K", "P", "x", "u", "info")
    dev = solve(w, H, first_only, want, torch.bfloat16)
    s = lqr.LqrSolver(n, n, H, batch)
    host = {k: w[k].cpu().pin_memory() for k in ("A", "B", "Q", "R", "x0")}
    out = lqr.alloc_outputs(n, n, H, N, "cpu", first_only=first_only, want=want, pin=True, dtype=torch.bfloat16)
    for k, v in out.items():
        v.fill_(-7 if k == "info" else 12345.0)
    flags = (lqr.TTC_OUT_FIRST_ONLY if first_only else 0) | lqr.TTC_OUT_BF16
    s.solve_host(host["A"], host["B"], host["Q"], host["R"], host["x0"], H, K=out.get("K"), P=out.get("P"), x=out.get("x"),
                 u=out.get("u"), info=out.get("info"), flags=flags)
    if n == 64:
        assert s.query(lqr.TTC_QUERY_LAST_LAUNCHES) > 1, "expected more than one slice"
    s.close()
    for k in want:
        assert torch.equal(out[k], dev[k].cpu()), k
