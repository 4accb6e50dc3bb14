"""Helpers shared by the GPU parity tests: run the CUDA library, run the oracle on the same
inputs (all or a sample of instances), and the error measure.

Error measure ("max relative error" of the target statement, made precise), per output tensor, per
instance and per time block t:
    err = max|gpu - ref| / max( max|ref block|, floor * max over t of max|ref| )
with floor = 1e-6 for K and P and floor = XU_FLOOR = 1e-4 for x and u; the reported figure is the maximum
over instances and t.  The closed loop contracts the state by many orders of magnitude over the horizon
(down to 3e-8 of |x_0| on the 16-state configuration, 1e-29 on the 32-state one) while
x_{t+1} = A x_t + B u_t cancels, so the rounding of ANY float32 computation is an absolute error on the
scale of the trajectory: tests/test_numerics_xu_error_measure.py shows a plain float32 recursion (LAPACK
Cholesky) at 2.2e-4 with a floor of 1e-6 and at 2.8e-5 with 1e-4, which is therefore the smallest decade
at which a 1e-4 bound is a property of the arithmetic and not of the sample.  The trajectory-normalised
figure (floor = 1: max over t of the error / max over t of the reference) is computed and returned too.
"""
import numpy as np
import torch

from oracle import lqr_oracle as orc
from paper_2603_09221_b200 import lqr


XU_FLOOR = 1e-4      # floor of the block-wise measure for x and u, relative to the largest block of the trajectory


def block_rel_err(gpu, ref, block_ndim, per_block=True, floor=1e-6):
    """gpu/ref: [M, T, ...block...] (or [M, ...block...] when there is no time axis)."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    if gpu.ndim == 1 + block_ndim:
        gpu, ref = gpu[:, None], ref[:, None]
    M, T = ref.shape[:2]
    g = gpu.reshape(M, T, -1)
    r = ref.reshape(M, T, -1)
    if not np.all(np.isfinite(g)):
        return float("inf")
    diff = np.abs(g - r).max(axis=2)
    blk = np.abs(r).max(axis=2)
    if not per_block:
        return float((diff.max(axis=1) / np.maximum(blk.max(axis=1), 1e-300)).max())
    lo = floor * blk.max(axis=1, keepdims=True)
    return float((diff / np.maximum(np.maximum(blk, lo), 1e-300)).max())


def run_gpu(w, method=lqr.TTC_RICCATI, want=("K", "P", "x", "u", "info"), first_only=None, math=lqr.TTC_MATH_AUTO,
            H=None, solver=None):
    """Solve workload ``w`` (tensors already on the GPU) through the C ABI."""
    n, m = w["n"], w["m"]
    H = w["H"] if H is None else H
    first_only = w["first_only"] if first_only is None else first_only
    N = int(np.prod(w["batch"]))
    dev = w["Q"].device
    own = solver is None
    if own:
        solver = lqr.LqrSolver(n, m, H, w["batch"], device=dev.index or 0, method=method, math=math)
    out = lqr.alloc_outputs(n, m, H, N, dev, first_only=first_only, want=want)
    for v in out.values():
        if v.dtype == torch.float32:
            v.fill_(123456.0)          # canary: every element must be overwritten
        else:
            v.fill_(-7)
    solver.solve(w["A"], w["B"], w["Q"], w["R"], w["x0"] if ("x" in want or "u" in want) else None, H,
                 K=out.get("K"), P=out.get("P"), x=out.get("x"), u=out.get("u"), info=out.get("info"),
                 flags=lqr.TTC_OUT_FIRST_ONLY if first_only else 0)
    torch.cuda.synchronize(dev)
    out["kernel"] = solver.query(lqr.TTC_QUERY_LAST_KERNEL)
    out["launches"] = solver.query(lqr.TTC_QUERY_LAST_LAUNCHES)
    assert solver.query(lqr.TTC_QUERY_DEVICE_ERROR) == 0, "a bounded wait inside the kernel ran out"
    if own:
        solver.close()
    return out


def gather_inputs(w, idx):
    """float64 numpy inputs of the instances ``idx`` (flat indices), one per row."""
    S, Hd, T = w["batch"]
    n, m = w["n"], w["m"]
    idx_t = torch.as_tensor(idx, device=w["Q"].device, dtype=torch.long)

    def sel(t, tail):
        full = t.expand((S, Hd, T) + tuple(tail)).reshape((S * Hd * T,) + tuple(tail))
        return full[idx_t].to(torch.float64).cpu().numpy()

    return (sel(w["A"], (n, n)), sel(w["B"], (n, m)), sel(w["Q"], (n, n)), sel(w["R"], (m, m)), sel(w["x0"], (n,)))


def run_oracle(w, idx=None, first_only=None, H=None, nthreads=0):
    N = int(np.prod(w["batch"]))
    if idx is None:
        idx = np.arange(N)
    A, B, Q, R, x0 = gather_inputs(w, idx)
    H = w["H"] if H is None else H
    first_only = w["first_only"] if first_only is None else first_only
    return orc.solve_batch(A, B, Q, R, x0, H, batch=(len(idx),), first_only=first_only, nthreads=nthreads)


def run_oracle_tv(w, idx=None, first_only=None, H=None, nthreads=0):
    """The time-varying oracle on the instances ``idx`` of a workload whose operands named in ``w["tv"]`` carry a
    time axis after the batch dimensions."""
    S, Hd, T = w["batch"]
    n, m = w["n"], w["m"]
    N = S * Hd * T
    H = w["H"] if H is None else H
    first_only = w["first_only"] if first_only is None else first_only
    idx_t = torch.as_tensor(np.arange(N) if idx is None else idx, device=w["Q"].device, dtype=torch.long)

    def sel(name, tail):
        t = w[name]
        if name in w["tv"]:
            t = t[..., :H, :, :]
            tail = (H,) + tuple(tail)
        full = t.expand((S, Hd, T) + tuple(tail)).reshape((N,) + tuple(tail))
        return full[idx_t].to(torch.float64).cpu().numpy()

    return orc.solve_batch_tv(sel("A", (n, n)), sel("B", (n, m)), sel("Q", (n, n)), sel("R", (m, m)), sel("Qf", (n, n)),
                              sel("x0", (n,)), H, (len(idx_t),), tv=w["tv"], first_only=first_only, nthreads=nthreads)


def compare(gpu, ref, idx, tol, names=("K", "P", "x", "u"), xu_floor=XU_FLOOR):
    """Returns {name: err} with the block-wise figure of every requested output and, for x and u, the
    trajectory-normalised one under "x_traj" / "u_traj"; asserts all of them within tol and info == 0.
    `xu_floor` replaces the floor of the block-wise x, u measure (1.0 = trajectory-normalised only)."""
    n_dims = {"K": 2, "P": 2, "x": 1, "u": 1}
    errs = {}
    sel = torch.as_tensor(idx, dtype=torch.long)
    for k in names:
        if k not in gpu or k not in ref:
            continue
        g = gpu[k].cpu()[sel].numpy()
        if k in ("x", "u"):
            errs[k] = block_rel_err(g, ref[k], n_dims[k], floor=xu_floor)
            errs[k + "_traj"] = block_rel_err(g, ref[k], n_dims[k], per_block=False)
        else:
            errs[k] = block_rel_err(g, ref[k], n_dims[k])
    if "info" in gpu:
        assert int(gpu["info"].cpu()[sel].abs().max()) == 0, "GPU reported failures on valid inputs"
    assert int(np.abs(ref["info"]).max()) == 0
    bad = {k: v for k, v in errs.items() if not (v <= tol)}
    assert not bad, "relative error above %g: %s (all: %s)" % (tol, bad, errs)
    return errs
