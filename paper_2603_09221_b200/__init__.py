"""B200-native batched finite-horizon LQR solve (the hot path of a Test-Time Control layer).

``lqr``       -- ctypes binding of the C ABI (``include/ttc_lqr.h``), CUDA only.
``workloads`` -- seeded synthetic inputs (no solver arithmetic).
``build``     -- nvcc build step of ``libttc_lqr.so``.
"""
from . import build, workloads  # noqa: F401

__all__ = ["build", "workloads", "lqr"]


def __getattr__(name):
    if name == "lqr":
        import importlib
        return importlib.import_module(".lqr", __name__)
    raise AttributeError(name)
