"""Long horizons with an open-loop unstable A (spectral radius 1.15).  The closed loop is well damped and the
Riccati recursion contracts symmetric errors, but an implementation that lets the rounding asymmetry of A'(P A) feed
back (the antisymmetric part E obeys E <- A'E A) loses P_0 after a few hundred steps.  Every backward kernel is
checked at H = 400 against the float64 oracle."""
import numpy as np
import pytest
import torch

from paper_2603_09221_b200 import lqr, workloads
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,batch,kernel", [(0, (1, 1, 6), "riccati_cta"), (1, (1, 2, 20), "riccati_warp"),
                                              (3, (1, 2, 10), "riccati_warp"), (4, (1, 2, 8), "riccati_umma"),
                                              (2, (1, 1, 8), "riccati_umma")])
def test_unstable_dynamics_long_horizon(cfg, batch, kernel):
    H = 400
    w = workloads.make_workload(cfg, device="cuda:0", batch=batch)
    w["A"] = (w["A"] * (1.15 / workloads.CONFIGS[cfg]["rho"])).contiguous()
    w["H"] = H
    N = int(np.prod(batch))
    for first_only in (True, False):
        names = ("P", "u") if first_only else ("K", "P", "x", "u")
        gpu = pu.run_gpu(w, want=names + ("info",), first_only=first_only, H=H)
        assert lqr.KERNEL_NAMES[gpu["kernel"]] == kernel
        ref = pu.run_oracle(w, first_only=first_only, H=H)
        # tf32 kernel: every gain is within the tolerance, but over 400 closed-loop steps the relative errors of the
        # gains compound in x_t while x_t itself decays far below the floor; its trajectory is compared as a whole
        # Its bound here is twice the configuration's: u_0 = -L^{-T} Z x_0 is formed from operands rounded to tf32
        # (2^-11) and amplified by the conditioning of S, which lands between 1e-2 and 2.5e-2 on these 400-step
        # problems whichever way the factorisation is organised; a loss of symmetry shows as an error of order one.
        tf32 = kernel == "riccati_umma"
        errs = pu.compare({k: gpu[k] for k in names + ("info",)}, ref, np.arange(N), w["tol"] * (2 if tf32 else 1),
                          names=names, xu_floor=1.0 if tf32 else pu.XU_FLOOR)
        print(cfg, first_only, errs)
        if "P" in names:
            P = gpu["P"].reshape((N, -1) + gpu["P"].shape[-2:])
            asym = float((P - P.transpose(-1, -2)).abs().max() / P.abs().max())
            assert asym <= (1e-6 if w["tol"] < 1e-3 else w["tol"] / 4), asym     # tf32 kernel: symmetrised every 8th step
