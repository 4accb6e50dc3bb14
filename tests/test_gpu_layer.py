"""GPU parity of the contextualised TTC-layer solve (ttc_lqr_solve_layer) against oracle/ttc_layer.py."""
import numpy as np
import pytest
import torch

from oracle import ttc_layer as lay
from paper_2603_09221_b200 import lqr, workloads
from tests import parity_util as pu

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_gpu(w, T, want_P=True, want_u=True):
    n, N = w["n"], w["N"]
    s = lqr.LqrSolver(n, n, max(T, 1), w["batch"])
    u1 = torch.full((N, n), 123456.0, device=DEV) if want_u else None
    P0 = torch.full((N, n, n), 123456.0, device=DEV) if want_P else None
    info = torch.full((N,), -7, dtype=torch.int32, device=DEV)
    s.solve_layer(*(w[k] for k in workloads.LAYER_KEYS), T, u1=u1, P0=P0, info=info)
    torch.cuda.synchronize()
    assert lqr.KERNEL_NAMES[s.query(lqr.TTC_QUERY_LAST_KERNEL)] == "ttc_layer"
    assert s.query(lqr.TTC_QUERY_LAST_LAUNCHES) == 1
    s.close()
    return u1, P0, info


def run_oracle(w, T, idx):
    sel = lambda k: w[k][torch.as_tensor(idx, device=w[k].device)].to(torch.float64).cpu().numpy()
    f64 = lambda k: w[k].to(torch.float64).cpu().numpy()
    return lay.solve_batch(sel("s_a"), sel("s_gamma_a"), sel("s_gamma_b"), sel("s_gamma_q"), sel("s_b"), sel("s_q"),
                           sel("s_qf"), sel("r_inv"), sel("h0"), f64("B_basis"), f64("Q_basis"), T)


def check(u1, P0, info, ref, idx, tol):
    sel = torch.as_tensor(idx)
    assert int(info.cpu()[sel].abs().max()) == 0 and int(np.abs(ref["info"]).max()) == 0
    errs = {}
    if P0 is not None:
        errs["P0"] = pu.block_rel_err(P0.cpu()[sel].numpy(), ref["P0"], 2)
    if u1 is not None:
        errs["u1"] = pu.block_rel_err(u1.cpu()[sel].numpy(), ref["u1"], 1)
    assert all(v <= tol for v in errs.values()), errs
    return errs


@pytest.mark.parametrize("key,batch,T", [("layer16", (1, 3, 7), 1), ("layer16", (2, 3, 9), 5), ("layer16", (1, 2, 33), 32),
                                         ("layer32", (1, 2, 5), 3), ("layer32", (2, 2, 6), 17), ("layer32", (1, 2, 40), 32)])
def test_layer_matches_oracle_on_every_instance(key, batch, T):
    """The full horizon at n = 32 is the case that shows a value matrix drifting away from symmetry: its diagonal
    A_t exceeds one, so an antisymmetric rounding residue doubles every few steps (1e-7 -> 1e-1 over 32 steps)."""
    w = workloads.make_layer_workload(key, device=DEV, batch=batch, seed=900 + T)
    u1, P0, info = run_gpu(w, T)
    idx = np.arange(w["N"])
    ref = run_oracle(w, T, idx)
    errs = check(u1, P0, info, ref, idx, 1e-4)
    print(key, batch, T, errs)
    assert not torch.any(u1 == 123456.0) and not torch.any(P0 == 123456.0) and not torch.any(info == -7)


def test_outputs_are_optional_and_independent():
    w = workloads.make_layer_workload("layer16", device=DEV, batch=(1, 2, 10), seed=31)
    u_all, P_all, _ = run_gpu(w, 6)
    u_only, none_P, _ = run_gpu(w, 6, want_P=False)
    none_u, P_only, _ = run_gpu(w, 6, want_u=False)
    assert none_P is None and none_u is None
    assert torch.equal(u_all, u_only) and torch.equal(P_all, P_only)


def test_unit_gamma_equals_the_dense_time_invariant_solver():
    """s_gamma = 0 and s_qf = s_q: the layer is a time-invariant LQR with A = I + diag(s_a); the dense solver must
    return the same first control (its P_0 additionally contains Q)."""
    w = workloads.make_layer_workload("layer16", device=DEV, batch=(1, 2, 8), seed=77)
    for k in ("s_gamma_a", "s_gamma_b", "s_gamma_q"):
        w[k] = torch.zeros_like(w[k])
    w["s_qf"] = w["s_q"].clone()
    T, n, N = 9, w["n"], w["N"]
    u1, P0, info = run_gpu(w, T)
    A = torch.diag_embed(1.0 + w["s_a"]).reshape(1, 2, 8, n, n)
    B = torch.einsum("ki,ijl->kjl", w["s_b"], w["B_basis"]).reshape(1, 2, 8, n, n).contiguous()
    Q = torch.einsum("ki,ijl->kjl", w["s_q"], w["Q_basis"]).reshape(1, 2, 8, n, n).contiguous()
    R = torch.diag_embed(1.0 / w["r_inv"]).reshape(1, 2, 8, n, n)
    s = lqr.LqrSolver(n, n, T, (1, 2, 8))
    out = lqr.alloc_outputs(n, n, T, N, DEV, first_only=True, want=("P", "u"))
    s.solve(A, B, Q, R, w["h0"].reshape(1, 2, 8, n), T, P=out["P"], u=out["u"], flags=lqr.TTC_OUT_FIRST_ONLY)
    torch.cuda.synchronize()
    s.close()
    assert float((out["u"] - u1).abs().max() / u1.abs().max()) < 2e-5
    assert float((out["P"] - Q.reshape(N, n, n) - P0).abs().max() / P0.abs().max()) < 2e-5


def test_non_positive_control_weight_is_reported_per_instance():
    w = workloads.make_layer_workload("layer16", device=DEV, batch=(1, 1, 6), seed=5)
    w["r_inv"][3, 2] = -0.05           # R_22 = -20: S = R + B'PB is not positive definite at the first step
    T = 4
    u1, P0, info = run_gpu(w, T)
    info = info.cpu().numpy()
    assert info[3] > 0 and (info[[0, 1, 2, 4, 5]] == 0).all()
    assert torch.isnan(u1[3]).all() and torch.isnan(P0[3]).all()
    good = np.array([0, 1, 2, 4, 5])
    ref = run_oracle(w, T, good)
    check(u1, P0, torch.as_tensor(info), ref, good, 1e-4)


def test_layer_full_size_on_sampled_instances():
    w = workloads.make_layer_workload("layer16", device=DEV)
    T = w["T"]
    u1, P0, info = run_gpu(w, T)
    assert int(info.abs().max()) == 0
    assert not torch.any(u1 == 123456.0) and not torch.any(P0 == 123456.0)
    idx = np.unique(np.concatenate([np.arange(0, w["N"], 509), [w["N"] - 1]]))
    ref = run_oracle(w, T, idx)
    print("layer16 sampled parity:", check(u1, P0, info, ref, idx, w["tol"]))
    Ps = P0[::97]
    assert float((Ps - Ps.transpose(-1, -2)).abs().max() / Ps.abs().max()) < 1e-5


def test_host_buffer_entry_point_pipelined_slices():
    """Enough instances for the host-buffer entry point to cut the batch into slices whose copies and solves overlap
    (ragged last slice): bit-equal to the device entry point, every output element written."""
    w = workloads.make_layer_workload("layer16", device=DEV, batch=(1, 5, 4001), seed=13)
    T, n, N = 6, w["n"], w["N"]
    u_d, P_d, info_d = run_gpu(w, T)
    s = lqr.LqrSolver(n, n, T, w["batch"])
    hin = [w[k].cpu().pin_memory() for k in workloads.LAYER_KEYS]
    u_h = torch.full((N, n), 7.0).pin_memory()
    P_h = torch.full((N, n, n), 7.0).pin_memory()
    info_h = torch.full((N,), -3, dtype=torch.int32).pin_memory()
    for _ in range(2):                                     # the staging buffers and events are reused
        s.solve_layer_host(*hin, T, u1=u_h, P0=P_h, info=info_h)
        assert s.query(lqr.TTC_QUERY_LAST_LAUNCHES) > 1, "expected more than one slice"
        assert torch.equal(u_h, u_d.cpu()) and torch.equal(P_h, P_d.cpu()) and torch.equal(info_h, info_d.cpu())
    s.close()


def test_layer_rejects_unsupported_shapes():
    s = lqr.LqrSolver(8, 8, 4, (1, 1, 4))
    w = workloads.make_layer_workload("layer16", device=DEV, batch=(1, 1, 4))
    with pytest.raises(Exception):
        s.solve_layer(*(w[k] for k in workloads.LAYER_KEYS), 2)
    s.close()


def test_host_buffer_entry_point_matches_device_entry_point():
    w = workloads.make_layer_workload("layer16", device=DEV, batch=(2, 3, 37), seed=12)
    T, n, N = 11, w["n"], w["N"]
    u_d, P_d, info_d = run_gpu(w, T)
    s = lqr.LqrSolver(n, n, T, w["batch"])
    hin = [w[k].cpu() for k in workloads.LAYER_KEYS]
    u_h = torch.full((N, n), 7.0).pin_memory()
    P_h = torch.full((N, n, n), 7.0).pin_memory()
    info_h = torch.full((N,), -3, dtype=torch.int32).pin_memory()
    s.solve_layer_host(*hin, T, u1=u_h, P0=P_h, info=info_h)
    assert s.query(lqr.TTC_QUERY_LAST_LAUNCHES) == 1
    assert torch.equal(u_h, u_d.cpu()) and torch.equal(P_h, P_d.cpu()) and torch.equal(info_h, info_d.cpu())
    # outputs are optional, pageable memory works, and the call can be repeated
    u2 = torch.empty((N, n))
    s.solve_layer_host(*hin, T, u1=u2)
    assert torch.equal(u2, u_d.cpu())
    s.close()
