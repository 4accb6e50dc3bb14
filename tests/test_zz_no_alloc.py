"""The allocation-free entry point (collected last on purpose).

Some callers cannot let the library call cudaMalloc when they need a solve: code running inside a
memory-pool callback, plugins whose host framework owns every device allocation, real-time loops.
``ttc_lqr_solve_first_noalloc`` serves them with a fixed scratch array inside the library.  This
test calls it through the C ABI twice in a row (the calls share the scratch, which keeps the
previous call's contents) and checks both results against the ordinary entry point.
"""
import numpy as np
import pytest
import torch

from paper_2603_09221_b200 import lqr, workloads
from tests import parity_util as pu

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _first_call_inputs(cfg, batch):
    w = workloads.make_workload(cfg, device=DEV, batch=batch)
    return w, int(np.prod(batch))


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    cases = [(1, (1, 8, 24)), (4, (1, 16, 4))]      # n=16/H=16 fp32 ; n=64/H=16 bf16, both fit the scratch
    prepared = []
    for cfg, batch in cases:
        w, N = _first_call_inputs(cfg, batch)
        ref = pu.run_gpu(w, method=lqr.TTC_SCAN, want=("P", "u", "info"), first_only=True)
        prepared.append((w, N, ref))
    for rep in range(2):                             # two rounds: scratch reused with stale contents
        for w, N, ref in prepared:
            n, m = w["n"], w["m"]
            P0 = torch.full((N, n, n), 123456.0, device=DEV)
            u0 = torch.full((N, m), 123456.0, device=DEV)
            info = torch.full((N,), -7, dtype=torch.int32, device=DEV)
            lqr.solve_first_noalloc(w["A"], w["B"], w["Q"], w["R"], w["x0"], w["H"], w["batch"], P0=P0, u0=u0, info=info)
            torch.cuda.synchronize()
            assert int(info.abs().max()) == 0
            tol = w["tol"]
            eP = pu.block_rel_err(P0.cpu().numpy(), ref["P"].cpu().numpy(), 2)
            eu = pu.block_rel_err(u0.cpu().numpy(), ref["u"].cpu().numpy(), 1, per_block=False)
            assert eP <= tol and eu <= tol, (rep, eP, eu)
            assert not torch.any(P0 == 123456.0) and not torch.any(u0 == 123456.0)


def test_noalloc_also_agrees_with_the_oracle():
    w, N = _first_call_inputs(1, (1, 8, 8))
    P0 = torch.empty((N, 16, 16), device=DEV)
    u0 = torch.empty((N, 16), device=DEV)
    info = torch.empty((N,), dtype=torch.int32, device=DEV)
    lqr.solve_first_noalloc(w["A"], w["B"], w["Q"], w["R"], w["x0"], w["H"], w["batch"], P0=P0, u0=u0, info=info)
    torch.cuda.synchronize()
    ref = pu.run_oracle(w, first_only=True)
    pu.compare({"P": P0, "u": u0, "info": info}, ref, np.arange(N), 1e-4, names=("P", "u"))


def test_noalloc_leaves_the_device_memory_untouched_and_runs_on_a_side_stream():
    """The property the entry point exists for: once the first call on the device has looked up the scratch address,
    a call changes the amount of free device memory by nothing.  Run on a non-default stream."""
    w, N = _first_call_inputs(1, (1, 8, 16))
    P0 = torch.empty((N, 16, 16), device=DEV)
    u0 = torch.empty((N, 16), device=DEV)
    info = torch.empty((N,), dtype=torch.int32, device=DEV)
    side = torch.cuda.Stream(device=DEV)
    args = (w["A"], w["B"], w["Q"], w["R"], w["x0"], w["H"], w["batch"])
    lqr.solve_first_noalloc(*args, P0=P0, u0=u0, info=info, stream=side)     # may be the address-resolving call
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info(0)[0]
    P0.fill_(123456.0)
    torch.cuda.synchronize()
    lqr.solve_first_noalloc(*args, P0=P0, u0=u0, info=info, stream=side)
    side.synchronize()
    assert torch.cuda.mem_get_info(0)[0] == free_before
    ref = pu.run_oracle(w, first_only=True)
    pu.compare({"P": P0, "u": u0, "info": info}, ref, np.arange(N), 1e-4, names=("P", "u"))


def test_noalloc_rejects_problems_beyond_its_scratch():
    w, N = _first_call_inputs(1, (4, 8, 128))        # 4096 instances x 16x16 floats = 4 MiB + status words
    P0 = torch.empty((N, 16, 16), device=DEV)
    with pytest.raises(lqr.TtcError) as ei:
        lqr.solve_first_noalloc(w["A"], w["B"], w["Q"], w["R"], None, w["H"], w["batch"], P0=P0)
    assert "scratch" in str(ei.value) and "INVALID_ARGUMENT" in str(ei.value)
