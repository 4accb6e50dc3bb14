"""Doubling for a P_0 / u_0-only request at n = m = 64 (configuration 4's shape): what it would buy.

The scan element of the time-invariant problem is e = (A, C = B R^{-1} B', J = Q); P_1 = e^(H-1) applied to Q by the
binary digits of H - 1, then one Riccati step gives P_0 and u_0.  Every solve inside `square` and `apply` can be put
in symmetric positive definite form (C = G G'; (I + J C)^{-1} J = J - Z'Z with Z = L^{-1} G'J, L L' = I + G'J G), so
that the blocked Cholesky the tensor-core kernel already has would serve -- at the price of one extra factorisation
(of C) per round.  This test restates both methods in numpy with the contractions' operands rounded to tf32 (what the
tensor-core kernel does) and records two facts:
  * accuracy is no obstacle: doubling reaches P_0, u_0 as well as the sequential recursion does;
  * the chain is: H = 16 needs 12 SPD factorisations by doubling against 16 sequentially, each doubling round with
    about three times the contractions of a Riccati step, all of them on per-instance operands (A_e, C_e, J_e, G_e
    and P: five 64 x 64 matrices per instance in shared memory instead of one), which would halve the number of
    instances an SM can keep in flight.  The sequential recursion is bound by the latency of its factorisation
    chain times the number of chains in flight, so 25 % fewer factorisations at half the chains is a loss.
"""
import numpy as np

from oracle import lqr_oracle as orc
from paper_2603_09221_b200 import workloads


def tf32(x):
    u = np.asarray(x, dtype=np.float32).view(np.uint32)
    return ((u + np.uint32(0x1000)) & np.uint32(0xFFFFE000)).view(np.float32)


def mm(a, b):
    return (tf32(a).astype(np.float64) @ tf32(b).astype(np.float64)).astype(np.float32)


def factor_tall(S, Yt):
    """L = chol(S), Z' = Y' L^{-T} at float32 grade (the kernel's factorisation is error-compensated)."""
    L = np.linalg.cholesky(S.astype(np.float64))
    return L.astype(np.float32), np.linalg.solve(L, Yt.T.astype(np.float64)).T.astype(np.float32)


def riccati_step(A, B, R, Q, P, count):
    V, T = mm(P, B), mm(P, A)
    S, Y = R + mm(B.T, V), mm(B.T, T)
    L, Zt = factor_tall(S, Y.T)
    count[0] += 1
    return Q + mm(A.T, T) - mm(Zt, Zt.T), L, Zt


def square(e, G, count):
    A, C, J = e
    eye = np.eye(len(A), dtype=np.float32)
    V = mm(J, G)
    _, Zt = factor_tall(eye + mm(G.T, V), V)
    count[0] += 1
    Jt = J - mm(Zt, Zt.T)                       # (I + J C)^{-1} J
    CJt = mm(C, Jt)
    A2 = mm(A, mm(eye - CJt, A))
    C2 = C + mm(mm(A, C - mm(CJt, C)), A.T)
    J2 = J + mm(mm(A.T, Jt), A)
    return A2, 0.5 * (C2 + C2.T), 0.5 * (J2 + J2.T)


def doubling_p1(A, B, R, Q, H, count):
    f = np.float32
    C = (B.astype(np.float64) @ np.linalg.solve(R.astype(np.float64), B.T.astype(np.float64))).astype(f)
    e, k, P = (A, 0.5 * (C + C.T), Q), H - 1, Q
    while k > 0:
        G = np.linalg.cholesky(e[1].astype(np.float64)).astype(f)
        count[0] += 1
        if k & 1:
            P = riccati_step(e[0], G, np.eye(len(A), dtype=f), e[2], P, count)[0]      # apply(e, P)
        k >>= 1
        if k > 0:
            e = square(e, G, count)
    return P


def test_doubling_is_accurate_in_tf32_but_saves_only_a_quarter_of_the_factorisations():
    batch, H, n = (1, 2, 2), 16, 64
    w = workloads.make_workload(4, device="cpu", batch=batch)
    d = workloads.to_float64_numpy(w)
    N = int(np.prod(batch))
    ref = orc.solve_batch(d["A"], d["B"], d["Q"], d["R"], d["x0"], H, batch=batch)
    P0r, u0r = ref["P"].reshape(N, H + 1, n, n)[:, 0], ref["u"].reshape(N, H, n)[:, 0]
    worst = {"riccati": [0.0, 0.0], "doubling": [0.0, 0.0]}
    for i in range(N):
        h = i // batch[2]
        A, B, R = (d[k][0, h, 0].astype(np.float32) for k in ("A", "B", "R"))
        Q, x0 = d["Q"].reshape(N, n, n)[i].astype(np.float32), d["x0"].reshape(N, n)[i]
        seq, dbl = [0], [0]
        P = Q
        for _ in range(H - 1):
            P = riccati_step(A, B, R, Q, P, seq)[0]
        for name, P1, cnt in (("riccati", P, seq), ("doubling", doubling_p1(A, B, R, Q, H, dbl), dbl)):
            P0, L, Zt = riccati_step(A, B, R, Q, P1, cnt)
            u0 = -np.linalg.solve(L.T.astype(np.float64), Zt.T.astype(np.float64)) @ x0
            worst[name][0] = max(worst[name][0], np.abs(P0 - P0r[i]).max() / np.abs(P0r[i]).max())
            worst[name][1] = max(worst[name][1], np.abs(u0 - u0r[i]).max() / np.abs(u0r[i]).max())
        assert seq[0] == 16 and dbl[0] == 12
    print("max rel err (P_0, u_0) with tf32 contractions:", worst)
    for name in worst:
        assert worst[name][0] < 2e-3 and worst[name][1] < 2e-2
    assert worst["doubling"][1] < 3 * worst["riccati"][1]
