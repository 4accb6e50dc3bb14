"""Why the fp32 kernels average P_t with its transpose: a float32 numpy restatement of the Riccati step (Prop. 3.1, in the
order the kernels use: V = P B, T = P A, S = R + B'V, Y = B'T, Z = L^{-1} Y, P <- Q + A'T - Z'Z), run on the time-varying
workload whose A_t = I + 0.1 G_t / sqrt(n) is open-loop unstable.  Without the averaging the antisymmetric rounding error
of A'T is propagated by A_t' (.) A_t and swamps P_0 at long horizons; with it the recursion stays at rounding level.  The
float64 oracle is the reference."""
import numpy as np

from oracle import lqr_oracle as orc
from paper_2603_09221_b200 import workloads


def fp32_recursion(A, B, Q, R, Qf, H, symmetrise):
    f = np.float32
    P = Qf.astype(f)
    for t in range(H - 1, -1, -1):
        a, b = A[t].astype(f), B[t].astype(f)
        V, T = P @ b, P @ a
        S = R[t].astype(f) + b.T @ V
        Y = b.T @ T
        L = np.linalg.cholesky(0.5 * (S + S.T)).astype(f)
        Z = np.linalg.solve(L, Y).astype(f)
        P = (Q[t].astype(f) + a.T @ T - Z.T @ Z).astype(f)
        if symmetrise:
            P = (f(0.5) * (P + P.T)).astype(f)
    return P


def test_antisymmetric_error_grows_without_the_averaging():
    H = 1024
    w = workloads.make_tv_workload("tv16", device="cpu", batch=(1, 1, 1), horizon=H)
    A, B, R = (w[k][0, 0, 0].numpy().astype(np.float64) for k in ("A", "B", "R"))
    Q, Qf, x0 = (w[k][0, 0, 0].numpy().astype(np.float64) for k in ("Q", "Qf", "x0"))
    assert max(np.abs(np.linalg.eigvals(A[t])).max() for t in range(0, H, 64)) > 1.05      # open-loop unstable
    K, P, x, u, info = orc.solve_tv(A, B, Q, R, Qf, x0, H)
    assert info == 0
    scale = np.abs(P[0]).max()
    plain = fp32_recursion(A, B, Q, R, Qf, H, symmetrise=False)
    kept = fp32_recursion(A, B, Q, R, Qf, H, symmetrise=True)
    assert np.abs(kept - P[0]).max() / scale < 5e-6
    assert np.abs(plain - P[0]).max() / scale > 1e-4                  # beyond the fp32 tolerance of the solver
    assert np.abs(plain - plain.T).max() > 100 * np.abs(kept - P[0]).max()     # and the damage is antisymmetric
