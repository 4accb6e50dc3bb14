"""The in-repo baseline: the row-normalised reverse symplectic product of Thm 3.3 (the paper's fused forward kernel)
on the contextualised layer's inputs.  At short horizons it must agree with the float64 layer oracle (which pins the
implementation: index mapping, Q_0 = 0, the Q_T override, the factorised Sigma_t, the pivoted solve of Y1 P = Y2 and
u_1 = -R_1^{-1} B_1' A_1^{-T} lambda_0); its float32 error then grows with the horizon, which is why the library's
layer solve is the backward recursion."""
import numpy as np
import pytest
import torch

from oracle import ttc_layer as lay
from paper_2603_09221_b200 import lqr, workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def errors(key, batch, T, baseline):
    w = workloads.make_layer_workload(key, device=DEV, batch=batch)
    n, N = w["n"], w["N"]
    s = lqr.LqrSolver(n, n, T, batch)
    u1 = torch.full((N, n), 7.0, device=DEV)
    P0 = torch.full((N, n, n), 7.0, device=DEV)
    info = torch.full((N,), -3, dtype=torch.int32, device=DEV)
    fn = s.solve_layer_sigma_baseline if baseline else s.solve_layer
    fn(*(w[k] for k in workloads.LAYER_KEYS), T, u1=u1, P0=P0, info=info)
    torch.cuda.synchronize()
    kernel = lqr.KERNEL_NAMES[s.query(lqr.TTC_QUERY_LAST_KERNEL)]
    s.close()
    f64 = lambda k: w[k].to(torch.float64).cpu().numpy()
    ref = lay.solve_batch(*(f64(k) for k in workloads.LAYER_KEYS[:9]), f64("B_basis"), f64("Q_basis"), T)
    eu = np.abs(u1.cpu().numpy() - ref["u1"]).max(axis=1) / np.abs(ref["u1"]).max(axis=1)
    eP = (np.abs(P0.cpu().numpy() - ref["P0"]).reshape(N, -1).max(axis=1) / np.abs(ref["P0"]).reshape(N, -1).max(axis=1))
    return eu, eP, info.cpu().numpy(), kernel


@pytest.mark.parametrize("key,batch", [("layer16", (1, 3, 21)), ("layer32", (1, 2, 9))])
def test_sigma_product_agrees_with_the_oracle_at_short_horizons(key, batch):
    for T, bound in ((1, 1e-5), (2, 1e-4)):
        eu, eP, info, kernel = errors(key, batch, T, baseline=True)
        assert kernel == "sigma_baseline" and int(np.abs(info).max()) == 0
        assert eu.max() <= bound and eP.max() <= bound, (T, eu.max(), eP.max())


def test_sigma_product_loses_accuracy_with_the_horizon_where_the_recursion_does_not():
    med = {}
    for T in (4, 16, 32):
        eu_s, eP_s, _, _ = errors("layer16", (1, 4, 32), T, baseline=True)
        eu_r, eP_r, info_r, _ = errors("layer16", (1, 4, 32), T, baseline=False)
        assert int(np.abs(info_r).max()) == 0 and max(eu_r.max(), eP_r.max()) <= 1e-5
        med[T] = float(np.nanmedian(eu_s))
    print("median relative error of u_1 by the sigma product:", med)
    assert med[4] < 1e-3 and med[16] > 1e-3 and med[32] > 1e-1
