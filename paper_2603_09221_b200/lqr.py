"""Thin ctypes binding of the C ABI in ``include/ttc_lqr.h``.

Argument marshalling only: every step of the solve runs in the CUDA kernels behind
``libttc_lqr.so``.  There is no CPU fallback; if the library is missing or no sm_100 device
is present, the calls raise.
PyTorch is used by callers for device memory and streams; this module only reads
``data_ptr()``, ``dtype``, ``shape`` and ``stride()`` of the tensors it is given.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

TTC_F32, TTC_BF16 = 0, 1
TTC_AUTO, TTC_RICCATI, TTC_SCAN = 0, 1, 2
TTC_MATH_AUTO, TTC_MATH_FP32, TTC_MATH_TF32 = 0, 1, 2
TTC_OUT_FIRST_ONLY = 1
TTC_OUT_BF16 = 2
TTC_QUERY_LAST_LAUNCHES, TTC_QUERY_WORKSPACE_BYTES, TTC_QUERY_LAST_KERNEL, TTC_QUERY_TOTAL_LAUNCHES = 1, 2, 3, 4
TTC_QUERY_DEVICE_ERROR = 5
KERNEL_NAMES = {7: "sigma_baseline", 6: "ttc_layer", 0: "none", 1: "riccati_cta", 2: "riccati_warp", 4: "scan", 5: "riccati_umma"}

EXPORTS = (
    "ttc_lqr_create", "ttc_lqr_solve", "ttc_lqr_solve_host", "ttc_lqr_destroy", "ttc_lqr_query",
    "ttc_lqr_status_string", "ttc_lqr_last_error", "ttc_lqr_solve_first_noalloc", "ttc_lqr_solve_tv",
    "ttc_lqr_solve_layer", "ttc_lqr_solve_layer_host", "ttc_lqr_solve_affine", "ttc_lqr_grad",
    "ttc_lqr_selftest_bounded_wait", "ttc_lqr_measure_fp32_peak", "ttc_lqr_solve_lowrank_q",
    "ttc_lqr_solve_layer_sigma_baseline", "ttc_lqr_layer_grad",
)
TTC_NOALLOC_SCRATCH_BYTES = 4 << 20


class ttc_operand(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("bstride", ctypes.c_int64 * 3)]


class ttc_layer_inputs(ctypes.Structure):
    _fields_ = [(k, ctypes.c_void_p) for k in ("s_a", "s_gamma_a", "s_gamma_b", "s_gamma_q", "s_b", "s_q", "s_qf",
                                               "r_inv", "h0", "B_basis", "Q_basis")] + [("r", ctypes.c_int32)]


LAYER_GRAD_KEYS = ("s_a", "s_gamma_a", "s_gamma_b", "s_gamma_q", "s_b", "s_q", "s_qf", "r_inv", "h0", "B_basis", "Q_basis")


class ttc_layer_grads(ctypes.Structure):
    _fields_ = [(k, ctypes.c_void_p) for k in LAYER_GRAD_KEYS]


class ttc_lqr_config(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int32), ("m", ctypes.c_int32), ("max_horizon", ctypes.c_int32),
                ("device", ctypes.c_int32), ("batch", ctypes.c_int64 * 3), ("method", ctypes.c_int32),
                ("math", ctypes.c_int32)]


class TtcError(RuntimeError):
    pass


_lib = None


def library_path() -> str:
    return _build.LIB


def load_library():
    """Load ``libttc_lqr.so`` (building it first if a source is newer).  Raises if that fails."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if not os.path.exists(path) or os.environ.get("TTC_LQR_REBUILD"):
        path = _build.build_library()
    lib = ctypes.CDLL(path)
    P = ctypes.POINTER
    lib.ttc_lqr_create.restype = ctypes.c_int
    lib.ttc_lqr_create.argtypes = [P(ttc_lqr_config), P(ctypes.c_void_p)]
    opp = P(ttc_operand)
    lib.ttc_lqr_solve.restype = ctypes.c_int
    lib.ttc_lqr_solve.argtypes = [ctypes.c_void_p, opp, opp, opp, opp, opp, ctypes.c_int32] + \
        [ctypes.c_void_p] * 5 + [ctypes.c_uint32, ctypes.c_void_p]
    lib.ttc_lqr_solve_lowrank_q.restype = ctypes.c_int
    lib.ttc_lqr_solve_lowrank_q.argtypes = [ctypes.c_void_p, opp, opp, opp, opp, ctypes.c_int32, ctypes.c_float, opp, opp,
                                            ctypes.c_int32] + [ctypes.c_void_p] * 5 + [ctypes.c_uint32, ctypes.c_void_p]
    lib.ttc_lqr_solve_tv.restype = ctypes.c_int
    lib.ttc_lqr_solve_tv.argtypes = [ctypes.c_void_p, opp, opp, opp, opp, P(ctypes.c_int64), opp, opp, ctypes.c_int32] + \
        [ctypes.c_void_p] * 5 + [ctypes.c_uint32, ctypes.c_void_p]
    lib.ttc_lqr_grad.restype = ctypes.c_int
    lib.ttc_lqr_grad.argtypes = [ctypes.c_void_p, opp, opp, opp, opp, P(ctypes.c_int64), opp, opp, ctypes.c_void_p,
                                 ctypes.c_int32] + [ctypes.c_void_p] * 9
    lib.ttc_lqr_solve_affine.restype = ctypes.c_int
    lib.ttc_lqr_solve_affine.argtypes = [ctypes.c_void_p, opp, opp, opp, opp, P(ctypes.c_int64), opp, opp, ctypes.c_int64,
                                         opp, ctypes.c_int32] + [ctypes.c_void_p] * 7 + [ctypes.c_uint32, ctypes.c_void_p]
    lib.ttc_lqr_solve_layer.restype = ctypes.c_int
    lib.ttc_lqr_solve_layer.argtypes = [ctypes.c_void_p, P(ttc_layer_inputs), ctypes.c_int32, ctypes.c_void_p,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    lib.ttc_lqr_solve_layer_sigma_baseline.restype = ctypes.c_int
    lib.ttc_lqr_solve_layer_sigma_baseline.argtypes = lib.ttc_lqr_solve_layer.argtypes
    lib.ttc_lqr_layer_grad.restype = ctypes.c_int
    lib.ttc_lqr_layer_grad.argtypes = [ctypes.c_void_p, P(ttc_layer_inputs), ctypes.c_int32, ctypes.c_void_p,
                                       P(ttc_layer_grads), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    lib.ttc_lqr_solve_layer_host.restype = ctypes.c_int
    lib.ttc_lqr_solve_layer_host.argtypes = [ctypes.c_void_p, P(ttc_layer_inputs), ctypes.c_int32, ctypes.c_void_p,
                                             ctypes.c_void_p, ctypes.c_void_p]
    lib.ttc_lqr_solve_host.restype = ctypes.c_int
    lib.ttc_lqr_solve_host.argtypes = [ctypes.c_void_p, opp, opp, opp, opp, opp, ctypes.c_int32] + \
        [ctypes.c_void_p] * 5 + [ctypes.c_uint32]
    lib.ttc_lqr_destroy.restype = ctypes.c_int
    lib.ttc_lqr_destroy.argtypes = [ctypes.c_void_p]
    lib.ttc_lqr_query.restype = ctypes.c_int
    lib.ttc_lqr_query.argtypes = [ctypes.c_void_p, ctypes.c_int32, P(ctypes.c_int64)]
    lib.ttc_lqr_status_string.restype = ctypes.c_char_p
    lib.ttc_lqr_status_string.argtypes = [ctypes.c_int]
    lib.ttc_lqr_last_error.restype = ctypes.c_char_p
    lib.ttc_lqr_last_error.argtypes = []
    lib.ttc_lqr_solve_first_noalloc.restype = ctypes.c_int
    lib.ttc_lqr_solve_first_noalloc.argtypes = [ctypes.c_int32, ctypes.c_int32, P(ctypes.c_int64), ctypes.c_int32,
                                                opp, opp, opp, opp, opp, ctypes.c_int32] + [ctypes.c_void_p] * 4
    lib.ttc_lqr_selftest_bounded_wait.restype = ctypes.c_int
    lib.ttc_lqr_selftest_bounded_wait.argtypes = [ctypes.c_int32, ctypes.c_int32, P(ctypes.c_int32)]
    lib.ttc_lqr_measure_fp32_peak.restype = ctypes.c_int
    lib.ttc_lqr_measure_fp32_peak.argtypes = [ctypes.c_int32, P(ctypes.c_double), P(ctypes.c_double)]
    _lib = lib
    return lib


def _check(status):
    if status != 0:
        lib = load_library()
        raise TtcError("%s: %s" % (lib.ttc_lqr_status_string(status).decode(), lib.ttc_lqr_last_error().decode()))


def _operand(t, tail_ndim, batch):
    """Describe tensor ``t`` (leading dims broadcastable to ``batch``, trailing ``tail_ndim``
    matrix/vector dims contiguous) as a ``ttc_operand``."""
    if t is None:
        return None
    if t.dtype == torch.float32:
        dt = TTC_F32
    elif t.dtype == torch.bfloat16:
        dt = TTC_BF16
    else:
        raise TypeError("operand dtype must be float32 or bfloat16, got %s" % t.dtype)
    lead = t.dim() - tail_ndim
    if lead > 3:
        raise ValueError("at most 3 batch dimensions")
    shape = (1,) * (3 - lead) + tuple(t.shape[:lead])
    strides = (0,) * (3 - lead) + tuple(t.stride()[:lead])
    exp = 1
    for d in range(t.dim() - 1, lead - 1, -1):
        if t.shape[d] != 1 and t.stride(d) != exp:
            raise ValueError("matrix dimensions of an operand must be contiguous (row-major)")
        exp *= t.shape[d]
    op = ttc_operand()
    op.ptr = t.data_ptr()
    op.dtype = dt
    op.reserved = 0
    for d in range(3):
        if shape[d] == batch[d]:
            op.bstride[d] = strides[d] if shape[d] > 1 else 0
        elif shape[d] == 1:
            op.bstride[d] = 0
        else:
            raise ValueError("operand batch shape %s does not broadcast to %s" % (shape, tuple(batch)))
    return op


class LqrSolver:
    """Owns one ``ttc_lqr_handle``.  ``batch`` is ``(seqs, heads, tokens)`` (shorter tuples are
    left-padded with 1)."""

    def __init__(self, n, m, max_horizon, batch, device=0, method=TTC_AUTO, math=TTC_MATH_AUTO):
        lib = load_library()
        batch = tuple(int(b) for b in batch)
        batch = (1,) * (3 - len(batch)) + batch
        cfg = ttc_lqr_config()
        cfg.n, cfg.m, cfg.max_horizon, cfg.device = n, m, max_horizon, device
        for d in range(3):
            cfg.batch[d] = batch[d]
        cfg.method, cfg.math = method, math
        self._h = ctypes.c_void_p()
        _check(lib.ttc_lqr_create(ctypes.byref(cfg), ctypes.byref(self._h)))
        self.n, self.m, self.batch, self.device = n, m, batch, device
        self.N = batch[0] * batch[1] * batch[2]

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            load_library().ttc_lqr_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def query(self, key):
        v = ctypes.c_int64()
        _check(load_library().ttc_lqr_query(self._h, key, ctypes.byref(v)))
        return v.value

    def _ops(self, A, B, Q, R, x0):
        ops = [_operand(A, 2, self.batch), _operand(B, 2, self.batch), _operand(Q, 2, self.batch),
               _operand(R, 2, self.batch), _operand(x0, 1, self.batch)]
        return [ctypes.byref(o) if o is not None else None for o in ops], ops

    @staticmethod
    def _ptr(t):
        return None if t is None else ctypes.c_void_p(t.data_ptr())

    def solve(self, A, B, Q, R, x0, H, K=None, P=None, x=None, u=None, info=None, flags=0, stream=None):
        """Enqueue ``ttc_lqr_solve`` on ``stream`` (a ``torch.cuda.Stream``; default: current)."""
        refs, keep = self._ops(A, B, Q, R, x0)
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        _check(load_library().ttc_lqr_solve(
            self._h, *refs, int(H), self._ptr(K), self._ptr(P), self._ptr(x), self._ptr(u), self._ptr(info),
            int(flags), ctypes.c_void_p(stream.cuda_stream)))

    def solve_lowrank_q(self, A, B, U, d, scale, R, x0, H, K=None, P=None, x=None, u=None, info=None, flags=0, stream=None):
        """Enqueue ``ttc_lqr_solve_lowrank_q``: as :meth:`solve` with ``Q = scale * U U' + diag(d)`` handed over as
        ``U [..batch.., n, rank]`` and ``d [..batch.., n]``."""
        ops = [_operand(A, 2, self.batch), _operand(B, 2, self.batch), _operand(U, 2, self.batch),
               _operand(d, 1, self.batch), _operand(R, 2, self.batch), _operand(x0, 1, self.batch)]
        ref = lambda o: ctypes.byref(o) if o is not None else None
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        _check(load_library().ttc_lqr_solve_lowrank_q(
            self._h, ref(ops[0]), ref(ops[1]), ref(ops[2]), ref(ops[3]), int(U.shape[-1]), ctypes.c_float(scale), ref(ops[4]),
            ref(ops[5]), int(H), self._ptr(K), self._ptr(P), self._ptr(x), self._ptr(u), self._ptr(info), int(flags),
            ctypes.c_void_p(stream.cuda_stream)))

    def solve_tv(self, A, B, Q, R, Qf, x0, H, tv=("A", "B", "Q", "R"), K=None, P=None, x=None, u=None, info=None,
                 flags=0, stream=None):
        """Enqueue ``ttc_lqr_solve_tv``.  Operands named in ``tv`` carry a time axis of length >= H right after
        their batch dimensions (``A [..batch.., H, n, n]``); the others are as for :meth:`solve`.  ``Qf`` is the
        terminal weight (may be None when Q is not time-varying)."""
        ops, tstride = [], (ctypes.c_int64 * 4)()
        for i, (name, t, tail) in enumerate((("A", A, 2), ("B", B, 2), ("Q", Q, 2), ("R", R, 2))):
            if name in tv:
                if t.shape[-3] < H:
                    raise ValueError("operand %s has %d time steps, H = %d" % (name, t.shape[-3], H))
                ops.append(_operand(t[..., 0, :, :], 2, self.batch))
                tstride[i] = t.stride(-3)
            else:
                ops.append(_operand(t, 2, self.batch))
                tstride[i] = 0
        oqf = _operand(Qf, 2, self.batch) if Qf is not None else None      # NULL: Q_f = Q (Q constant in time)
        ox = _operand(x0, 1, self.batch)
        ref = lambda o: ctypes.byref(o) if o is not None else None
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        _check(load_library().ttc_lqr_solve_tv(
            self._h, ref(ops[0]), ref(ops[1]), ref(ops[2]), ref(ops[3]), tstride, ref(oqf), ref(ox), int(H),
            self._ptr(K), self._ptr(P), self._ptr(x), self._ptr(u), self._ptr(info), int(flags),
            ctypes.c_void_p(stream.cuda_stream)))

    def solve_affine(self, A, B, Q, R, Qf, r, x0, H, tv=("A", "B", "Q", "R", "r"), K=None, kff=None, P=None, pvec=None,
                     x=None, u=None, info=None, flags=0, stream=None):
        """Enqueue ``ttc_lqr_solve_affine`` (linear control cost ``r_t'u_t``; Prop. A.1).  As :meth:`solve_tv`; ``r`` is
        ``[..batch.., H, m]`` when ``"r"`` is in ``tv``, else ``[..batch.., m]``.  ``kff [N, H, m]`` receives the
        feed-forward terms, ``pvec [N, H + 1, n]`` (``[N, n]`` with first-only) the linear value terms."""
        ops, tstride = [], (ctypes.c_int64 * 4)()
        for i, (name, t) in enumerate((("A", A), ("B", B), ("Q", Q), ("R", R))):
            if name in tv:
                if t.shape[-3] < H:
                    raise ValueError("operand %s has %d time steps, H = %d" % (name, t.shape[-3], H))
                ops.append(_operand(t[..., 0, :, :], 2, self.batch))
                tstride[i] = t.stride(-3)
            else:
                ops.append(_operand(t, 2, self.batch))
                tstride[i] = 0
        if "r" in tv:
            if r.shape[-2] < H:
                raise ValueError("operand r has %d time steps, H = %d" % (r.shape[-2], H))
            orr, rst = _operand(r[..., 0, :], 1, self.batch), r.stride(-2)
        else:
            orr, rst = _operand(r, 1, self.batch), 0
        oqf = _operand(Qf, 2, self.batch) if Qf is not None else None      # NULL: Q_f = Q (Q constant in time)
        ox = _operand(x0, 1, self.batch)
        ref = lambda o: ctypes.byref(o) if o is not None else None
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        _check(load_library().ttc_lqr_solve_affine(
            self._h, ref(ops[0]), ref(ops[1]), ref(ops[2]), ref(ops[3]), tstride, ref(oqf), ref(orr), int(rst), ref(ox),
            int(H), self._ptr(K), self._ptr(kff), self._ptr(P), self._ptr(pvec), self._ptr(x), self._ptr(u),
            self._ptr(info), int(flags), ctypes.c_void_p(stream.cuda_stream)))

    def grad(self, A, B, Q, R, Qf, x0, g, H, tv=("A", "B", "Q", "R"), dA=None, dB=None, dQ=None, dQf=None, dR=None,
             dx0=None, u0=None, info=None, stream=None):
        """Enqueue ``ttc_lqr_grad`` (Thm 3.2): gradients of a loss of the first control ``u_0*`` given ``g = dl/du_0*``
        (``[N, m]`` float32).  Operands as for :meth:`solve_tv`.  Outputs, each optional: ``dA [N, H, n, n]``,
        ``dB [N, H, n, m]``, ``dQ [N, H, n, n]``, ``dQf [N, n, n]``, ``dR [N, H, m, m]``, ``dx0 [N, n]``, ``u0 [N, m]``,
        ``info [N]`` (int32)."""
        ops, tstride = [], (ctypes.c_int64 * 4)()
        for i, (name, t) in enumerate((("A", A), ("B", B), ("Q", Q), ("R", R))):
            if name in tv:
                if t.shape[-3] < H:
                    raise ValueError("operand %s has %d time steps, H = %d" % (name, t.shape[-3], H))
                ops.append(_operand(t[..., 0, :, :], 2, self.batch))
                tstride[i] = t.stride(-3)
            else:
                ops.append(_operand(t, 2, self.batch))
                tstride[i] = 0
        oqf = _operand(Qf, 2, self.batch) if Qf is not None else None      # NULL: Q_f = Q (Q constant in time)
        ox = _operand(x0, 1, self.batch)
        if tuple(g.shape) != (self.N, self.m) or g.dtype != torch.float32 or not g.is_contiguous():
            raise ValueError("g must be a contiguous float32 tensor of shape (%d, %d)" % (self.N, self.m))
        ref = lambda o: ctypes.byref(o) if o is not None else None
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        _check(load_library().ttc_lqr_grad(
            self._h, ref(ops[0]), ref(ops[1]), ref(ops[2]), ref(ops[3]), tstride, ref(oqf), ref(ox), self._ptr(g), int(H),
            self._ptr(dA), self._ptr(dB), self._ptr(dQ), self._ptr(dQf), self._ptr(dR), self._ptr(dx0), self._ptr(u0),
            self._ptr(info), ctypes.c_void_p(stream.cuda_stream)))

    def _layer_inputs(self, tensors, host):
        s_a, s_gamma_a, s_gamma_b, s_gamma_q, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis = tensors
        r = int(B_basis.shape[0])
        n, N = self.n, self.N
        per_n = dict(s_a=s_a, s_gamma_a=s_gamma_a, s_gamma_b=s_gamma_b, s_gamma_q=s_gamma_q, r_inv=r_inv, h0=h0)
        per_r = dict(s_b=s_b, s_q=s_q, s_qf=s_qf)
        inp = ttc_layer_inputs()
        for name, t in list(per_n.items()) + list(per_r.items()) + [("B_basis", B_basis), ("Q_basis", Q_basis)]:
            want = (N, n) if name in per_n else (N, r) if name in per_r else (r, n, n)
            if host:
                placed = t.device.type == "cpu"
            else:
                placed = t.device.type == "cuda" and (t.device.index or 0) == self.device
            if tuple(t.shape) != want or t.dtype != torch.float32 or not t.is_contiguous() or not placed:
                raise ValueError("%s must be a contiguous float32 tensor of shape %s on %s" %
                                 (name, want, "the host" if host else "cuda:%d" % self.device))
            setattr(inp, name, t.data_ptr())
        inp.r = r
        return inp

    def solve_layer(self, s_a, s_gamma_a, s_gamma_b, s_gamma_q, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis, T,
                    u1=None, P0=None, info=None, stream=None):
        """Enqueue ``ttc_lqr_solve_layer``: contextualised TTC-layer evaluation.  Per-instance tensors are
        ``[N, n]`` (``s_b, s_q, s_qf``: ``[N, r]``), the bases ``[r, n, n]``; all float32, contiguous, on the
        solver's device.  ``u1 [N, n]``, ``P0 [N, n, n]``, ``info [N]`` (int32) are written if given."""
        inp = self._layer_inputs((s_a, s_gamma_a, s_gamma_b, s_gamma_q, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis), False)
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        _check(load_library().ttc_lqr_solve_layer(
            self._h, ctypes.byref(inp), int(T), self._ptr(u1), self._ptr(P0), self._ptr(info),
            ctypes.c_void_p(stream.cuda_stream)))

    def solve_layer_sigma_baseline(self, s_a, s_gamma_a, s_gamma_b, s_gamma_q, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis, T,
                                   u1=None, P0=None, info=None, stream=None):
        """``ttc_lqr_solve_layer_sigma_baseline``: the same layer evaluation by the row-normalised reverse symplectic
        product (a baseline whose float32 error grows with the horizon); arguments as :meth:`solve_layer`."""
        inp = self._layer_inputs((s_a, s_gamma_a, s_gamma_b, s_gamma_q, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis), False)
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        _check(load_library().ttc_lqr_solve_layer_sigma_baseline(
            self._h, ctypes.byref(inp), int(T), self._ptr(u1), self._ptr(P0), self._ptr(info),
            ctypes.c_void_p(stream.cuda_stream)))

    def layer_grad(self, s_a, s_gamma_a, s_gamma_b, s_gamma_q, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis, T, g,
                   grads, u1=None, info=None, stream=None):
        """Enqueue ``ttc_lqr_layer_grad``: gradients of a loss of the layer output ``u_1*`` given ``g = dl/du_1*``
        (``[N, n]`` float32).  ``grads`` maps any of ``LAYER_GRAD_KEYS`` to an output tensor shaped like the input of
        that name (the basis gradients are summed over the instances)."""
        inp = self._layer_inputs((s_a, s_gamma_a, s_gamma_b, s_gamma_q, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis), False)
        out = ttc_layer_grads()
        for k in LAYER_GRAD_KEYS:
            t = grads.get(k)
            if t is not None and (t.dtype != torch.float32 or not t.is_contiguous()):
                raise ValueError("gradient output %s must be a contiguous float32 tensor" % k)
            setattr(out, k, None if t is None else t.data_ptr())
        if tuple(g.shape) != (self.N, self.n) or g.dtype != torch.float32 or not g.is_contiguous():
            raise ValueError("g must be a contiguous float32 tensor of shape (%d, %d)" % (self.N, self.n))
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        _check(load_library().ttc_lqr_layer_grad(
            self._h, ctypes.byref(inp), int(T), self._ptr(g), ctypes.byref(out), self._ptr(u1), self._ptr(info),
            ctypes.c_void_p(stream.cuda_stream)))

    def solve_layer_host(self, s_a, s_gamma_a, s_gamma_b, s_gamma_q, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis, T,
                         u1=None, P0=None, info=None):
        """``ttc_lqr_solve_layer_host``: all tensors live in host memory; returns when the results are there."""
        inp = self._layer_inputs((s_a, s_gamma_a, s_gamma_b, s_gamma_q, s_b, s_q, s_qf, r_inv, h0, B_basis, Q_basis), True)
        _check(load_library().ttc_lqr_solve_layer_host(
            self._h, ctypes.byref(inp), int(T), self._ptr(u1), self._ptr(P0), self._ptr(info)))

    def solve_host(self, A, B, Q, R, x0, H, K=None, P=None, x=None, u=None, info=None, flags=0):
        """``ttc_lqr_solve_host``: all tensors live in host memory; returns when the results are there."""
        refs, keep = self._ops(A, B, Q, R, x0)
        _check(load_library().ttc_lqr_solve_host(
            self._h, *refs, int(H), self._ptr(K), self._ptr(P), self._ptr(x), self._ptr(u), self._ptr(info),
            int(flags)))


def alloc_outputs(n, m, H, N, device, first_only=False, want=("K", "P", "x", "u", "info"), pin=False,
                  dtype=torch.float32):
    """Allocate output tensors of the documented shapes (torch owns the memory); ``dtype=torch.bfloat16`` for calls
    made with ``TTC_OUT_BF16``."""
    kw = dict(device=device)
    if pin and str(device) == "cpu":
        kw["pin_memory"] = True
    out = {}
    if "K" in want:
        out["K"] = torch.empty((N, H, m, n), dtype=dtype, **kw)
    if "P" in want:
        out["P"] = torch.empty((N, n, n) if first_only else (N, H + 1, n, n), dtype=dtype, **kw)
    if "x" in want:
        out["x"] = torch.empty((N, H + 1, n), dtype=dtype, **kw)
    if "u" in want:
        out["u"] = torch.empty((N, m) if first_only else (N, H, m), dtype=dtype, **kw)
    if "info" in want:
        out["info"] = torch.empty((N,), dtype=torch.int32, **kw)
    return out


def measure_fp32_peak(device=0):
    """``ttc_lqr_measure_fp32_peak``: measured FP32 FMA rate of the device in TFLOP/s as ``(scalar, packed)``."""
    a, b = ctypes.c_double(), ctypes.c_double()
    _check(load_library().ttc_lqr_measure_fp32_peak(int(device), ctypes.byref(a), ctypes.byref(b)))
    return a.value, b.value


def selftest_bounded_wait(poll_limit=4096, device=0):
    """``ttc_lqr_selftest_bounded_wait``: runs the give-up branch of the kernels' bounded barrier wait on a
    barrier nothing arrives on; returns 1 when the timeout was reported through the error word."""
    out = ctypes.c_int32(-1)
    _check(load_library().ttc_lqr_selftest_bounded_wait(int(device), int(poll_limit), ctypes.byref(out)))
    return out.value


def solve_first_noalloc(A, B, Q, R, x0, H, batch, P0=None, u0=None, info=None, device=0, stream=None):
    """``ttc_lqr_solve_first_noalloc``: P_0 / u_0 by the scan method without any device allocation
    by the library -- for callers that may not allocate (allocator callbacks, hosts that own all
    device memory, real-time loops).  The scratch is a fixed ``TTC_NOALLOC_SCRATCH_BYTES`` array
    inside the library; problems that need more are rejected with ``TtcError``.  Calls share that
    array, so do not let two of them overlap on the GPU."""
    lib = load_library()
    batch = tuple(int(b) for b in batch)
    batch = (1,) * (3 - len(batch)) + batch
    n, m = B.shape[-2], B.shape[-1]
    ops = [_operand(A, 2, batch), _operand(B, 2, batch), _operand(Q, 2, batch), _operand(R, 2, batch),
           _operand(x0, 1, batch)]
    refs = [ctypes.byref(o) if o is not None else None for o in ops]
    if stream is None:
        stream = torch.cuda.current_stream(device)
    barr = (ctypes.c_int64 * 3)(*batch)
    ptr = LqrSolver._ptr
    _check(lib.ttc_lqr_solve_first_noalloc(n, m, barr, device, *refs, int(H), ptr(P0), ptr(u0), ptr(info),
                                           ctypes.c_void_p(stream.cuda_stream)))
