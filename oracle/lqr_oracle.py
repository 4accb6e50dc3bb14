"""ctypes front end of the float64 CPU oracle (``lqr_oracle.c``).

TEST INFRASTRUCTURE ONLY: used by the tests, the smoke check and the benchmark's
CPU-baseline leg.  It imports nothing from the CUDA package and the CUDA package
imports nothing from here.

The arithmetic lives in ``lqr_oracle.c`` (Prop. 3.1 / Alg. 1 of the paper, written
out as plain loops in float64).  This module only compiles that file with gcc,
marshals numpy arrays and expands broadcast batch dimensions into per-instance
offsets.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lqr_oracle.c")
_LIB = os.path.join(_HERE, "liblqr_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile ``lqr_oracle.c`` into ``liblqr_oracle.so`` next to it (gcc, OpenMP)."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int64)
        lib.lqr_oracle_solve.restype = ctypes.c_int
        lib.lqr_oracle_solve.argtypes = [ctypes.c_int] * 3 + [dp] * 9 + [ctypes.c_int]
        lib.lqr_oracle_solve_batch.restype = ctypes.c_int
        lib.lqr_oracle_solve_batch.argtypes = (
            [ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int]
            + [dp, ip] * 5
            + [dp] * 4
            + [ctypes.POINTER(ctypes.c_int32), ctypes.c_int, ctypes.c_int]
        )
        lib.lqr_oracle_solve_tv.restype = ctypes.c_int
        lib.lqr_oracle_solve_tv.argtypes = [ctypes.c_int] * 3 + [dp, ctypes.c_int64] * 4 + [dp] * 6 + [ctypes.c_int]
        lib.lqr_oracle_solve_affine.restype = ctypes.c_int
        lib.lqr_oracle_solve_affine.argtypes = [ctypes.c_int] * 3 + [dp, ctypes.c_int64] * 5 + [dp] * 8
        lib.lqr_oracle_solve_batch_tv.restype = ctypes.c_int
        lib.lqr_oracle_solve_batch_tv.argtypes = (
            [ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int]
            + [dp, ip, ctypes.c_int64] * 4
            + [dp, ip] * 2
            + [dp] * 4
            + [ctypes.POINTER(ctypes.c_int32), ctypes.c_int, ctypes.c_int]
        )
        _lib = lib
    return _lib


def _dptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def solve(A, B, Q, R, x0, H, first_only=False):
    """One instance.  Returns ``(K, P, x, u, info)`` as float64 arrays.

    Shapes: ``K [H,m,n]``, ``P [H+1,n,n]`` (``[n,n]`` if ``first_only``), ``x [H+1,n]``,
    ``u [H,m]`` (``[m]`` if ``first_only``).
    """
    A, B, Q, R, x0 = map(_f64, (A, B, Q, R, x0))
    n, m = B.shape
    assert A.shape == (n, n) and Q.shape == (n, n) and R.shape == (m, m) and x0.shape == (n,)
    K = np.empty((H, m, n))
    P = np.empty((n, n) if first_only else (H + 1, n, n))
    x = np.empty((H + 1, n))
    u = np.empty((m,) if first_only else (H, m))
    info = _load().lqr_oracle_solve(
        n, m, H, _dptr(A), _dptr(B), _dptr(Q), _dptr(R), _dptr(x0),
        _dptr(K), _dptr(P), _dptr(x), _dptr(u), int(first_only))
    return K, P, x, u, info


def _offsets(arr, batch, tail):
    """Element offsets of every instance of a (possibly broadcast) batched operand."""
    arr = _f64(arr)
    assert arr.shape[-len(tail):] == tuple(tail), (arr.shape, tail)
    lead = arr.shape[: arr.ndim - len(tail)]
    lead = (1,) * (len(batch) - len(lead)) + tuple(lead)
    arr = arr.reshape(lead + tuple(tail))
    view = np.broadcast_to(arr, tuple(batch) + tuple(tail))
    off = np.zeros(tuple(batch), dtype=np.int64)
    for d, nb in enumerate(batch):
        shape = [1] * len(batch)
        shape[d] = nb
        off = off + (np.arange(nb, dtype=np.int64) * (view.strides[d] // 8)).reshape(shape)
    return arr, np.ascontiguousarray(off.reshape(-1))


def solve_batch(A, B, Q, R, x0, H, batch=None, first_only=False, nthreads=0,
                want=("K", "P", "x", "u")):
    """Many instances.  Operands carry leading batch dimensions that broadcast to
    ``batch`` (a tuple; default: the broadcast of all operands' leading dims).

    Returns a dict with the requested outputs (float64, leading dim ``N = prod(batch)``),
    ``info`` (int32 per instance) and ``threads`` (OpenMP threads used).
    """
    B_ = np.asarray(B)
    n, m = B_.shape[-2:]
    if batch is None:
        batch = np.broadcast_shapes(
            np.asarray(A).shape[:-2], B_.shape[:-2], np.asarray(Q).shape[:-2],
            np.asarray(R).shape[:-2], np.asarray(x0).shape[:-1])
    batch = tuple(int(b) for b in batch)
    N = int(np.prod(batch)) if batch else 1
    A_, oA = _offsets(A, batch, (n, n))
    B_, oB = _offsets(B, batch, (n, m))
    Q_, oQ = _offsets(Q, batch, (n, n))
    R_, oR = _offsets(R, batch, (m, m))
    x_, ox = _offsets(x0, batch, (n,))
    out = {}
    K = np.empty((N, H, m, n)) if "K" in want else None
    P = (np.empty((N, n, n) if first_only else (N, H + 1, n, n))) if "P" in want else None
    x = np.empty((N, H + 1, n)) if "x" in want else None
    u = (np.empty((N, m) if first_only else (N, H, m))) if "u" in want else None
    info = np.zeros(N, dtype=np.int32)
    ip = ctypes.POINTER(ctypes.c_int64)
    used = _load().lqr_oracle_solve_batch(
        N, n, m, H,
        _dptr(A_), oA.ctypes.data_as(ip), _dptr(B_), oB.ctypes.data_as(ip),
        _dptr(Q_), oQ.ctypes.data_as(ip), _dptr(R_), oR.ctypes.data_as(ip),
        _dptr(x_), ox.ctypes.data_as(ip),
        _dptr(K), _dptr(P), _dptr(x), _dptr(u),
        info.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), int(first_only), int(nthreads))
    for k, v in (("K", K), ("P", P), ("x", x), ("u", u)):
        if v is not None:
            out[k] = v
    out["info"] = info
    out["threads"] = used
    return out


def solve_tv(A, B, Q, R, Qf, x0, H, first_only=False):
    """One time-varying instance (Definition A.1 / Prop. A.1 with A_t, B_t, Q_t, R_t, terminal weight Qf).

    ``A`` is ``[H,n,n]`` or ``[n,n]`` (the same at every t); likewise ``B [H,n,m]``, ``Q [H,n,n]``,
    ``R [H,m,m]``.  Index t of each is the matrix of step t: ``x_{t+1} = A_t x_t + B_t u_t``, stage cost
    ``x_t'Q_t x_t + u_t'R_t u_t``, terminal cost ``x_H'Qf x_H``.  Returns ``(K, P, x, u, info)``.
    """
    A, B, Q, R, Qf, x0 = map(_f64, (A, B, Q, R, Qf, x0))
    n, m = B.shape[-2:]
    strides = []
    for a, tail in ((A, (n, n)), (B, (n, m)), (Q, (n, n)), (R, (m, m))):
        assert a.shape in (tail, (H,) + tail), (a.shape, tail)
        strides.append(0 if a.ndim == 2 else tail[0] * tail[1])
    assert Qf.shape == (n, n) and x0.shape == (n,)
    K = np.empty((H, m, n))
    P = np.empty((n, n) if first_only else (H + 1, n, n))
    x = np.empty((H + 1, n))
    u = np.empty((m,) if first_only else (H, m))
    info = _load().lqr_oracle_solve_tv(
        n, m, H, _dptr(A), strides[0], _dptr(B), strides[1], _dptr(Q), strides[2], _dptr(R), strides[3],
        _dptr(Qf), _dptr(x0), _dptr(K), _dptr(P), _dptr(x), _dptr(u), int(first_only))
    return K, P, x, u, info


def solve_batch_tv(A, B, Q, R, Qf, x0, H, batch, tv=("A", "B", "Q", "R"), first_only=False, nthreads=0,
                   want=("K", "P", "x", "u")):
    """Many time-varying instances.  Operands named in ``tv`` carry a time axis of length ``H`` right after
    their (broadcastable) batch dimensions, e.g. ``A [..batch.., H, n, n]``; the others are ``[..batch.., n, n]``.
    Returns the same dict as :func:`solve_batch`."""
    n, m = np.asarray(B).shape[-2:]
    batch = tuple(int(b) for b in batch)
    N = int(np.prod(batch))
    ops, offs, strides = {}, {}, {}
    for name, arr, tail in (("A", A, (n, n)), ("B", B, (n, m)), ("Q", Q, (n, n)), ("R", R, (m, m))):
        full_tail = ((H,) + tail) if name in tv else tail
        ops[name], offs[name] = _offsets(arr, batch, full_tail)
        strides[name] = tail[0] * tail[1] if name in tv else 0
    Qf_, oQf = _offsets(Qf, batch, (n, n))
    x_, ox = _offsets(x0, batch, (n,))
    K = np.empty((N, H, m, n)) if "K" in want else None
    P = (np.empty((N, n, n) if first_only else (N, H + 1, n, n))) if "P" in want else None
    x = np.empty((N, H + 1, n)) if "x" in want else None
    u = (np.empty((N, m) if first_only else (N, H, m))) if "u" in want else None
    info = np.zeros(N, dtype=np.int32)
    ip = ctypes.POINTER(ctypes.c_int64)
    args = []
    for name in ("A", "B", "Q", "R"):
        args += [_dptr(ops[name]), offs[name].ctypes.data_as(ip), strides[name]]
    used = _load().lqr_oracle_solve_batch_tv(
        N, n, m, H, *args, _dptr(Qf_), oQf.ctypes.data_as(ip), _dptr(x_), ox.ctypes.data_as(ip),
        _dptr(K), _dptr(P), _dptr(x), _dptr(u),
        info.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), int(first_only), int(nthreads))
    out = {k: v for k, v in (("K", K), ("P", P), ("x", x), ("u", u)) if v is not None}
    out["info"] = info
    out["threads"] = used
    return out


def solve_affine(A, B, Q, R, r, Qf, x0, H):
    """One instance with a linear control cost (Definition A.1 with ``r_t``; Prop. A.1): stage cost
    ``1/2 (x_t'Q_t x_t + u_t'R_t u_t) + r_t'u_t``, terminal cost ``1/2 x_H'Qf x_H``.  Operands as for
    :func:`solve_tv`; ``r`` is ``[H, m]`` or ``[m]``.  Returns a dict with ``K [H,m,n]``, ``k [H,m]`` (feed-forward:
    ``u_t = K_t x_t + k_t``), ``P [H+1,n,n]``, ``p [H+1,n]``, ``x [H+1,n]``, ``u [H,m]``, ``info``."""
    A, B, Q, R, r, Qf, x0 = map(_f64, (A, B, Q, R, r, Qf, x0))
    n, m = B.shape[-2:]
    strides = []
    for a, tail in ((A, (n, n)), (B, (n, m)), (Q, (n, n)), (R, (m, m)), (r, (m,))):
        assert a.shape in (tail, (H,) + tail), (a.shape, tail)
        strides.append(0 if a.ndim == len(tail) else int(np.prod(tail)))
    assert Qf.shape == (n, n) and x0.shape == (n,)
    K = np.empty((H, m, n)); k = np.empty((H, m)); P = np.empty((H + 1, n, n)); p = np.empty((H + 1, n))
    x = np.empty((H + 1, n)); u = np.empty((H, m))
    info = _load().lqr_oracle_solve_affine(
        n, m, H, _dptr(A), strides[0], _dptr(B), strides[1], _dptr(Q), strides[2], _dptr(R), strides[3],
        _dptr(r), strides[4], _dptr(Qf), _dptr(x0), _dptr(K), _dptr(k), _dptr(P), _dptr(p), _dptr(x), _dptr(u))
    return dict(K=K, k=k, P=P, p=p, x=x, u=u, info=info)
