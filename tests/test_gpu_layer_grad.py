"""GPU parity of ttc_lqr_layer_grad (gradients of the contextualised layer's output with respect to the coefficient
vectors, R^{-1}, h_0 and the shared bases) against the float64 oracle oracle/ttc_layer_grad.py, which is pinned by
finite differences of the forward layer oracle."""
import numpy as np
import pytest
import torch

from oracle import ttc_layer_grad as og
from paper_2603_09221_b200 import lqr, workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PER_INSTANCE = lqr.LAYER_GRAD_KEYS[:9]


def run_both(key, batch, T, seed=None, want=lqr.LAYER_GRAD_KEYS, with_info=True):
    w = workloads.make_layer_workload(key, device=DEV, batch=batch, seed=seed)
    n, N = w["n"], w["N"]
    gen = torch.Generator(device=DEV)
    gen.manual_seed(1234 + N + T)
    g = torch.randn((N, n), generator=gen, device=DEV)
    s = lqr.LqrSolver(n, n, T, batch)
    grads = {k: torch.full_like(w[k], 777.0) for k in want}
    u1 = torch.full((N, n), 777.0, device=DEV)
    info = torch.full((N,), -5, dtype=torch.int32, device=DEV) if with_info else None
    s.layer_grad(*(w[k] for k in workloads.LAYER_KEYS), T, g, grads, u1=u1, info=info)
    torch.cuda.synchronize()
    launches = s.query(lqr.TTC_QUERY_LAST_LAUNCHES)
    s.close()
    f64 = lambda t: t.to(torch.float64).cpu().numpy()
    refs = [og.grad(*(f64(w[k][i]) for k in workloads.LAYER_KEYS[:9]), f64(w["B_basis"]), f64(w["Q_basis"]), T, f64(g[i]))
            for i in range(N)]
    return w, grads, u1, info, refs, launches


def rel(a, b):
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))


@pytest.mark.parametrize("key,batch,T", [("layer16", (1, 3, 7), 6), ("layer16", (2, 2, 9), 1), ("layer16", (1, 1, 5), 32),
                                         ("layer32", (1, 2, 5), 9), ("layer32", (1, 1, 3), 2)])
def test_every_gradient_matches_the_oracle(key, batch, T):
    w, grads, u1, info, refs, launches = run_both(key, batch, T)
    N = w["N"]
    assert launches == 4                                   # backward pass, vectors + reductions, two basis reductions
    assert int(info.abs().max()) == 0
    for i in range(N):
        assert rel(u1[i].cpu().numpy(), refs[i]["u1"]) <= 1e-4
        for k in PER_INSTANCE:
            got = grads[k][i].double().cpu().numpy()
            assert np.all(np.isfinite(got)), k
            # relative to the largest entry of that gradient vector of the instance
            assert np.abs(got - refs[i][k]).max() <= 1e-4 * max(np.abs(refs[i][k]).max(), 1e-7), (k, i, got, refs[i][k])
    for k in ("B_basis", "Q_basis"):                       # shared by the instances: the oracle's per-instance terms are summed
        ref = sum(r_[k] for r_ in refs)
        assert rel(grads[k].double().cpu().numpy(), ref) <= 1e-4, k
    Qg = grads["Q_basis"]
    assert float((Qg - Qg.transpose(1, 2)).abs().max()) <= 1e-5 * float(Qg.abs().max())


def test_two_column_backward_pass_at_a_batch_that_fills_the_machine():
    """More than 2368 instances at n = 16: the backward pass runs with two columns per lane (the kernel the benchmark's
    layer16 gradients use).  Sampled instances against the oracle; the basis gradients, which sum over every instance,
    against a second call in which the same instances go through the one-column kernel in two halves."""
    key, batch, T = "layer16", (1, 4, 640), 5
    w = workloads.make_layer_workload(key, device=DEV, batch=batch, seed=77)
    n, N = w["n"], w["N"]
    gen = torch.Generator(device=DEV)
    gen.manual_seed(99)
    g = torch.randn((N, n), generator=gen, device=DEV)

    def call(lo, hi):
        s = lqr.LqrSolver(n, n, T, (1, 1, hi - lo))
        grads = {k: torch.full_like(w[k] if k in ("B_basis", "Q_basis") else w[k][lo:hi], 777.0) for k in lqr.LAYER_GRAD_KEYS}
        u1 = torch.full((hi - lo, n), 777.0, device=DEV)
        info = torch.full((hi - lo,), -5, dtype=torch.int32, device=DEV)
        ins = [w[k] if k in ("B_basis", "Q_basis") else w[k][lo:hi].contiguous() for k in workloads.LAYER_KEYS]
        s.layer_grad(*ins, T, g[lo:hi].contiguous(), grads, u1=u1, info=info)
        torch.cuda.synchronize()
        s.close()
        return grads, u1, info

    full, u_full, info = call(0, N)
    assert int(info.abs().max()) == 0
    halves = [call(0, N // 2), call(N // 2, N)]
    f64 = lambda t: t.to(torch.float64).cpu().numpy()
    for i in range(0, N, 107):
        ref = og.grad(*(f64(w[k][i]) for k in workloads.LAYER_KEYS[:9]), f64(w["B_basis"]), f64(w["Q_basis"]), T, f64(g[i]))
        assert rel(u_full[i].cpu().numpy(), ref["u1"]) <= 1e-4
        for k in PER_INSTANCE:
            got = full[k][i].double().cpu().numpy()
            assert np.abs(got - ref[k]).max() <= 1e-4 * max(np.abs(ref[k]).max(), 1e-7), (k, i)
    for k in PER_INSTANCE:
        both = torch.cat([halves[0][0][k], halves[1][0][k]])
        assert float((full[k] - both).abs().max()) <= 1e-4 * float(both.abs().max()), k
    for k in ("B_basis", "Q_basis"):
        both = halves[0][0][k].double() + halves[1][0][k].double()
        assert float((full[k].double() - both).abs().max()) <= 1e-4 * float(both.abs().max()), k


def test_partial_requests_and_no_info():
    w, grads, u1, info, refs, launches = run_both("layer16", (1, 2, 6), 5, want=("s_a", "h0", "s_q"), with_info=False)
    assert launches == 2 and set(grads) == {"s_a", "h0", "s_q"}
    for i in range(w["N"]):
        for k in grads:
            assert np.abs(grads[k][i].double().cpu().numpy() - refs[i][k]).max() <= 1e-4 * max(np.abs(refs[i][k]).max(), 1e-7)


def test_failed_instance_gets_nan_and_is_left_out_of_the_basis_gradients():
    key, batch, T = "layer16", (1, 1, 6), 4
    w = workloads.make_layer_workload(key, device=DEV, batch=batch)
    n, N = w["n"], w["N"]
    w["r_inv"] = w["r_inv"].clone()
    w["r_inv"][3] = -1.0                                   # R = diag(1 / r_inv) negative: R + B'PB loses definiteness
    w["s_q"] = w["s_q"].clone()
    w["s_q"][3] = 0.0
    w["s_qf"] = w["s_qf"].clone()
    w["s_qf"][3] = 0.0
    g = torch.randn((N, n), generator=torch.Generator(device=DEV).manual_seed(9), device=DEV)
    s = lqr.LqrSolver(n, n, T, batch)
    grads = {k: torch.zeros_like(w[k]) for k in lqr.LAYER_GRAD_KEYS}
    info = torch.zeros((N,), dtype=torch.int32, device=DEV)
    s.layer_grad(*(w[k] for k in workloads.LAYER_KEYS), T, g, grads, info=info)
    torch.cuda.synchronize()
    s.close()
    assert int(info[3]) > 0 and int((info != 0).sum()) == 1
    for k in PER_INSTANCE:
        assert bool(torch.isnan(grads[k][3]).all()), k
        assert bool(torch.isfinite(grads[k][[0, 1, 2, 4, 5]]).all()), k
    f64 = lambda t: t.to(torch.float64).cpu().numpy()
    good = [i for i in range(N) if i != 3]
    refs = [og.grad(*(f64(w[k][i]) for k in workloads.LAYER_KEYS[:9]), f64(w["B_basis"]), f64(w["Q_basis"]), T, f64(g[i])) for i in good]
    for k in ("B_basis", "Q_basis"):
        assert bool(torch.isfinite(grads[k]).all())
        assert rel(grads[k].double().cpu().numpy(), sum(r_[k] for r_ in refs)) <= 1e-4, k
