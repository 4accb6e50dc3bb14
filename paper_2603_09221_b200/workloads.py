"""Seeded synthetic inputs shaped like TTC-layer LQR workloads.

This module only draws random numbers and assembles input tensors; it contains none
of the solver's arithmetic and is the one module that both the CUDA path's callers
(tests, bench) and the CPU oracle's callers may use.

Batch layout is ``[seq][head][token]``; instance index ``i = (s*heads + h)*tokens + k``.
Operands shared by a head have size-1 ``seq`` and ``token`` dimensions.

Recipe (one seed per configuration, ``260309221 + c``):
  A = G * rho / rho(G), G_ij ~ N(0,1), rho(G) = max |eigenvalue|   (float64 on the host)
  B_ij ~ N(0, 1/n)            R = M M'/m + 0.1 I  (M m x m Gaussian)
  Q = L L'/n + 0.1 I  (L n x n Gaussian)        x0 ~ N(0, I)
  configuration 4: Q = U U'/8 + diag(d), U n x 8 Gaussian, d_i ~ U[0.05, 0.2]
A, B, R are float32.  Q and x0 are float32, or rounded to bfloat16 (round to nearest
even, element-wise, which keeps Q symmetric) where the configuration says so.
"""
from __future__ import annotations

import numpy as np
import torch

SEED0 = 260309221

CONFIGS = {
    0: dict(name="cfg0_tiny_n8_H8", batch=(1, 1, 64), n=8, m=8, H=8, rho=0.9,
            per_instance_system=True, q_dtype="f32", q_kind="full", first_only=False, tol=1e-4),
    1: dict(name="cfg1_small_n16_H16", batch=(4, 8, 128), n=16, m=16, H=16, rho=0.9,
            per_instance_system=False, q_dtype="f32", q_kind="full", first_only=False, tol=1e-4),
    2: dict(name="cfg2_medium_n64_H8_bf16", batch=(4, 8, 2048), n=64, m=64, H=8, rho=0.9,
            per_instance_system=False, q_dtype="bf16", q_kind="full", first_only=False, tol=2e-2),
    3: dict(name="cfg3_long_n32_H64", batch=(1, 16, 1024), n=32, m=32, H=64, rho=0.98,
            per_instance_system=False, q_dtype="f32", q_kind="full", first_only=False, tol=1e-4),
    4: dict(name="cfg4_large_n64_H16_bf16_first", batch=(2, 16, 4096), n=64, m=64, H=16, rho=0.9,
            per_instance_system=False, q_dtype="bf16", q_kind="lowrank8", first_only=True, tol=2e-2),
}


# Time-varying workload shaped like the paper's TTC layer: state dimension 16, 16 heads, horizon 32.  Dynamics and
# control cost belong to the head and change with the time index, state cost / terminal weight / initial state
# belong to the token.  Stand-in for the layer's learned parameters (near-identity A_t, diagonal-dominant R_t,
# rank-16 Q_t): A_t = I + 0.1 G_t / sqrt(n), B_t ~ N(0, 1/n), R_t = diag(U[0.5, 1.5]) + 0.05 M_t M_t'/m,
# Q_t = L_t L_t'/n + 0.05 I, Q_f likewise, x0 ~ N(0, I).
TV_CONFIGS = {
    "tv16": dict(name="tv16_ttc_layer_d16_T32", batch=(4, 16, 1024), n=16, m=16, H=32, q_dtype="f32",
                 first_only=True, tol=1e-4, tv=("A", "B", "Q", "R")),
    # the time-varying problem at d = 32 per head (a quarter of the tokens: the same bytes of Q_t)
    "tv32": dict(name="tv32_ttc_layer_d32_T32", batch=(4, 16, 256), n=32, m=32, H=32, q_dtype="f32",
                 first_only=True, tol=1e-4, tv=("A", "B", "Q", "R")),
    # the same problem, differentiated: gradients of a loss of u_0* with respect to every A_t, B_t, Q_t, R_t, Q_f, x_0
    "grad16": dict(name="grad16_ttc_layer_d16_T32", batch=(4, 16, 1024), n=16, m=16, H=32, q_dtype="f32",
                   first_only=True, tol=1e-4, tv=("A", "B", "Q", "R"), grad=True),
}


def make_tv_workload(key="tv16", device="cpu", batch=None, seed=None, chunk=4096, horizon=None):
    """Inputs of a time-varying configuration: ``A, B, R [1,Hd,1,H,...]`` (float32, per head and time index),
    ``Q [S,Hd,T,H,n,n]``, ``Qf [S,Hd,T,n,n]``, ``x0 [S,Hd,T,n]`` plus the configuration fields."""
    c = dict(TV_CONFIGS[key])
    if batch is not None:
        c["batch"] = tuple(int(b) for b in batch)
    if horizon is not None:
        c["H"] = int(horizon)
    S, Hd, T = c["batch"]
    n, m, H = c["n"], c["m"], c["H"]
    seed = SEED0 + 100 if seed is None else seed
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    rn = lambda *shape: torch.randn(shape, generator=gen, device=device)
    eye_n, eye_m = torch.eye(n, device=device), torch.eye(m, device=device)
    A = eye_n + 0.1 * rn(1, Hd, 1, H, n, n) / n ** 0.5
    B = rn(1, Hd, 1, H, n, m) / n ** 0.5
    M = rn(1, Hd, 1, H, m, m)
    R = torch.diag_embed(0.5 + torch.rand((1, Hd, 1, H, m), generator=gen, device=device)) + 0.05 * M @ M.transpose(-1, -2) / m
    R = 0.5 * (R + R.transpose(-1, -2))
    N = S * Hd * T
    Q = torch.empty((N, H, n, n), dtype=torch.float32, device=device)
    for s0 in range(0, N, chunk):
        cnt = min(chunk, N - s0)
        L = rn(cnt, H, n, n)
        q = L @ L.transpose(-1, -2) / n + 0.05 * eye_n
        Q[s0:s0 + cnt] = 0.5 * (q + q.transpose(-1, -2))
    Lf = rn(N, n, n)
    Qf = Lf @ Lf.transpose(-1, -2) / n + 0.05 * eye_n
    Qf = 0.5 * (Qf + Qf.transpose(-1, -2))
    x0 = rn(N, n)
    c.update(A=A.contiguous(), B=B.contiguous(), R=R.contiguous(), Q=Q.reshape(S, Hd, T, H, n, n),
             Qf=Qf.reshape(S, Hd, T, n, n), x0=x0.reshape(S, Hd, T, n), seed=seed)
    return c


def _system(rng, n, m, rho):
    G = rng.standard_normal((n, n))
    A = G * (rho / np.max(np.abs(np.linalg.eigvals(G))))
    B = rng.standard_normal((n, m)) / np.sqrt(n)
    M = rng.standard_normal((m, m))
    R = M @ M.T / m + 0.1 * np.eye(m)
    return A, B, 0.5 * (R + R.T)


def make_workload(cfg_id, device="cpu", batch=None, seed=None, chunk=8192):
    """Build the inputs of configuration ``cfg_id`` (optionally with a smaller/larger
    ``batch = (seqs, heads, tokens)``).

    Returns a dict: ``A [*,n,n]``, ``B [*,n,m]``, ``R [*,m,m]`` (float32), ``Q [S,Hd,T,n,n]`` and
    ``x0 [S,Hd,T,n]`` (float32 or bfloat16) as torch tensors on ``device``, plus the
    configuration fields (``n, m, H, batch, first_only, tol, name``).
    """
    c = dict(CONFIGS[cfg_id])
    if batch is not None:
        c["batch"] = tuple(int(b) for b in batch)
    S, Hd, T = c["batch"]
    n, m = c["n"], c["m"]
    seed = SEED0 + cfg_id if seed is None else seed
    rng = np.random.default_rng(seed)

    if c["per_instance_system"]:
        sys_shape = (S, Hd, T)
    else:
        sys_shape = (1, Hd, 1)
    nsys = int(np.prod(sys_shape))
    As, Bs, Rs = zip(*[_system(rng, n, m, c["rho"]) for _ in range(nsys)])
    to32 = lambda lst, shp: torch.from_numpy(
        np.stack(lst).astype(np.float32).reshape(sys_shape + shp)).to(device)
    A, B, R = to32(As, (n, n)), to32(Bs, (n, m)), to32(Rs, (m, m))

    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    N = S * Hd * T
    qdt = torch.bfloat16 if c["q_dtype"] == "bf16" else torch.float32
    Q = torch.empty((N, n, n), dtype=qdt, device=device)
    low = c["q_kind"] != "full"
    Uf = torch.empty((N, n, 8), dtype=qdt, device=device) if low else None       # the factors themselves, for callers that
    df = torch.empty((N, n), dtype=qdt, device=device) if low else None          # hand Q over as U U'/8 + diag(d)
    eye = torch.eye(n, device=device)
    for s0 in range(0, N, chunk):
        cnt = min(chunk, N - s0)
        if c["q_kind"] == "full":
            L = torch.randn((cnt, n, n), generator=gen, device=device)
            q = L @ L.transpose(1, 2) / n + 0.1 * eye
        else:
            U = torch.randn((cnt, n, 8), generator=gen, device=device)
            d = 0.05 + 0.15 * torch.rand((cnt, n), generator=gen, device=device)
            q = U @ U.transpose(1, 2) / 8 + torch.diag_embed(d)
            Uf[s0:s0 + cnt] = U.to(qdt)
            df[s0:s0 + cnt] = d.to(qdt)
        q = 0.5 * (q + q.transpose(1, 2))
        Q[s0:s0 + cnt] = q.to(qdt)
    x0 = torch.randn((N, n), generator=gen, device=device).to(qdt)
    c.update(A=A, B=B, R=R, Q=Q.reshape(S, Hd, T, n, n), x0=x0.reshape(S, Hd, T, n),
             seed=seed, cfg_id=cfg_id)
    if low:
        c.update(U=Uf.reshape(S, Hd, T, n, 8), d=df.reshape(S, Hd, T, n), q_scale=1.0 / 8)
    return c


def to_float64_numpy(w):
    """Widen a workload's tensors exactly to float64 numpy arrays (what the oracle reads)."""
    return {k: w[k].detach().to("cpu").to(torch.float64).numpy() for k in ("A", "B", "Q", "R", "x0")}


# Contextualised TTC-layer workload (Contextualization paragraph): state dimension d = 16 per head, 16 heads,
# r = 16 basis matrices shared by all heads, planning horizon T = 32; one instance per (sequence, head, token).
# The coefficient layers' outputs are drawn directly (trained weights are not available): s_A ~ 0.3 N(0,1),
# s_Gamma* = softplus(N(0,1) - 2) (decay rates mostly in (0.05, 0.5)), s_B ~ N(0, 1/r), s_Q, s_Qf = softplus(N(0,1)) / r,
# r_inv = softplus(N(0,1)) + 0.5, h0 ~ N(0, I); B^(i) ~ N(0, 1/d), Q^(i) = Qc Qc' / sqrt(d) with Qc ~ N(0, 1).
LAYER_CONFIGS = {
    "layer16": dict(name="layer16_ctx_d16_r16_T32", batch=(4, 16, 1024), n=16, r=16, T=32, tol=1e-4),
    "layer32": dict(name="layer32_ctx_d32_r16_T32", batch=(2, 8, 1024), n=32, r=16, T=32, tol=1e-4),
}


def make_layer_workload(key="layer16", device="cpu", batch=None, seed=None):
    """Inputs of ``ttc_lqr_solve_layer`` for a contextualised-layer configuration (float32 tensors, instance-major)."""
    c = dict(LAYER_CONFIGS[key])
    if batch is not None:
        c["batch"] = tuple(int(b) for b in batch)
    N = c["batch"][0] * c["batch"][1] * c["batch"][2]
    n, r = c["n"], c["r"]
    seed = SEED0 + 200 if seed is None else seed
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    rn = lambda *shape: torch.randn(shape, generator=gen, device=device)
    sp = torch.nn.functional.softplus
    Qc = rn(r, n, n)
    c.update(
        s_a=(0.3 * rn(N, n)).contiguous(), s_gamma_a=sp(rn(N, n) - 2.0), s_gamma_b=sp(rn(N, n) - 2.0),
        s_gamma_q=sp(rn(N, n) - 2.0), s_b=rn(N, r) / r ** 0.5, s_q=sp(rn(N, r)) / r, s_qf=sp(rn(N, r)) / r,
        r_inv=sp(rn(N, n)) + 0.5, h0=rn(N, n), B_basis=rn(r, n, n) / n ** 0.5,
        Q_basis=(Qc @ Qc.transpose(-1, -2) / n ** 0.5).contiguous(), seed=seed, N=N)
    return c


LAYER_KEYS = ("s_a", "s_gamma_a", "s_gamma_b", "s_gamma_q", "s_b", "s_q", "s_qf", "r_inv", "h0", "B_basis", "Q_basis")
