"""How the n = m = 64 tensor-core kernel gets the gains K_t = -(R + B'PB)^{-1} B'PA (Eq. 4) without a backward solve.

The kernel factors the tall matrix [S; Y'] (S = R + B'PB, Y = B'PA) by a right-looking blocked Cholesky with 8-wide
panels: every row is one thread, a panel's rows are substituted with the diagonal block and ONE rank-8 update
G -= panel * panel[0:64]' is applied to all 128 rows and all 64 columns.  It leaves L (S = L L') and Z' = Y' L^{-T}.
With gains requested, rows 0..63 do not stop at their diagonal block: to the right of the diagonal their row of the
work matrix is the unused upper triangle of S, which the updates keep equal to the lower one and which the row's own
panel brings to zero; from there on the row is continued as row r of X = L^{-T} (in the diagonal panel the operand row is
L[r, p] + e_r L_d^{-T}, afterwards whatever the row reads back, substituted).  Because rows 0..63 of the panel are also
the second operand of the update, the updates subtract Z'[n, p] X[r, p]' from column r of the rows of Z' once that
column has been consumed: after the last panel the columns of rows 64..127 hold -Z' X' = -Z' L^{-1} = K_t'.

This file restates that scheme in numpy (float64, no rounding) and checks
  * that it returns L, Z' and K_t' exactly (against numpy's Cholesky and solve);
  * that it depends on the upper triangle of S being the mirror of the lower one: an antisymmetric perturbation of
    relative size 1e-3 in the upper triangle (what single-pass tf32 contractions leave there) changes L and Z' not
    at all but K_t' by the same order, which is why the kernel mirrors the lower triangle first.
"""
import numpy as np

N, PW = 64, 8


def fsub(x, Ld):
    """x (row vectors) <- x Ld^{-T} for a lower-triangular 8 x 8 block."""
    return np.linalg.solve(Ld, x.T).T


def factor_with_gains(G):
    """G = [S; Y'] (128 x 64).  Returns L, Z' and the final contents of rows 64..127 (the gains, transposed)."""
    G = G.copy()
    L = np.zeros((N, N))
    Zt = np.zeros((N, N))
    for p in range(N // PW):
        c0 = PW * p
        cols = slice(c0, c0 + PW)
        Ld = np.linalg.cholesky(np.tril(G[cols, cols]) + np.tril(G[cols, cols], -1).T)     # diagonal block: lower triangle only
        panel = np.zeros((2 * N, PW))
        for r in range(2 * N):
            v = fsub(G[r:r + 1, cols], Ld)[0]
            if r >= N:                                   # a row of Z'
                Zt[r - N, cols] = v
                panel[r] = v
            elif r >= c0 + PW:                           # a row of L still to come
                L[r, cols] = v
                panel[r] = v
            elif r >= c0:                                # its diagonal panel: L ends here, X = L^{-T} starts
                v[r - c0 + 1:] = 0.0
                L[r, cols] = v
                e = np.zeros(PW)
                e[r - c0] = 1.0
                panel[r] = v + fsub(e[None, :], Ld)[0]
            else:                                        # finished row: what it reads back is its row of X, substituted
                panel[r] = v
        G -= panel @ panel[:N].T                         # every row, every column; rows 0..63 are the second operand
    return L, Zt, G[N:]


def problem(seed):
    rng = np.random.default_rng(seed)
    M = rng.standard_normal((N, N))
    S = M @ M.T / N + 0.2 * np.eye(N)
    Y = rng.standard_normal((N, N))
    return S, Y


def test_updates_collect_the_transposed_gains():
    S, Y = problem(1)
    L, Zt, Kt = factor_with_gains(np.vstack([S, Y.T]))
    Lref = np.linalg.cholesky(S)
    assert np.abs(L - Lref).max() < 1e-12
    assert np.abs(Zt - np.linalg.solve(Lref, Y).T).max() < 1e-11
    K = -np.linalg.solve(S, Y)                           # Eq. 4 with S = R + B'PB, Y = B'PA
    assert np.abs(Kt - K.T).max() < 1e-10 * np.abs(K).max()


def test_an_asymmetric_upper_triangle_goes_straight_into_the_gains():
    S, Y = problem(2)
    rng = np.random.default_rng(3)
    E = np.triu(rng.standard_normal((N, N)), 1) * 1e-3 * np.abs(S).mean()
    K = -np.linalg.solve(S, Y)
    Lref = np.linalg.cholesky(S)
    L, Zt, Kt = factor_with_gains(np.vstack([S + E, Y.T]))          # lower triangle untouched
    assert np.abs(L - Lref).max() < 1e-12 and np.abs(Zt - np.linalg.solve(Lref, Y).T).max() < 1e-11
    err = np.abs(Kt - K.T).max() / np.abs(K).max()
    assert 1e-5 < err < 1e-1, err                        # the perturbation reaches the gains at its own order
    Sm = np.tril(S + E) + np.tril(S + E, -1).T           # the kernel's remedy: mirror the lower triangle first
    _, _, Kt2 = factor_with_gains(np.vstack([Sm, Y.T]))
    assert np.abs(Kt2 - K.T).max() < 1e-10 * np.abs(K).max()
