"""CPU-side checks of the C-ABI library: it builds for sm_100a, loads, exports every symbol the
header declares, and refuses to work without a CUDA device (no CPU fallback)."""
import ctypes
import os
import re

import pytest
import torch

from paper_2603_09221_b200 import build, lqr

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(ttc_\w+)\s*\(", text)
    return sorted(set(names))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build_library()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    decl = declared_functions()
    assert len(decl) >= 7
    for name in decl:
        assert hasattr(lib, name), "header declares %s but the library does not export it" % name
    assert set(lqr.EXPORTS) <= set(decl)


def test_status_strings():
    lib = lqr.load_library()
    assert lib.ttc_lqr_status_string(0) == b"TTC_OK"
    assert lib.ttc_lqr_status_string(-1) == b"TTC_STATUS_INVALID_ARGUMENT"
    assert lib.ttc_lqr_status_string(-99) == b"TTC_STATUS_UNKNOWN"


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful on a machine without a GPU")
def test_no_cpu_fallback_without_a_device():
    with pytest.raises(lqr.TtcError):
        lqr.LqrSolver(8, 8, 8, (1, 1, 4))


def test_create_rejects_bad_config_before_touching_the_device():
    for kw in (dict(n=0), dict(m=65), dict(max_horizon=0), dict(batch=(0, 1, 1)), dict(method=7), dict(math=9)):
        args = dict(n=8, m=8, max_horizon=4, batch=(1, 1, 4))
        args.update(kw)
        with pytest.raises(lqr.TtcError) as ei:
            lqr.LqrSolver(**args)
        assert "INVALID_ARGUMENT" in str(ei.value)


def test_operand_marshalling_strides_and_broadcast():
    A = torch.zeros((1, 3, 1, 4, 4))
    Q = torch.zeros((2, 3, 5, 4, 4))
    x0 = torch.zeros((2, 3, 5, 4), dtype=torch.bfloat16)
    oa = lqr._operand(A, 2, (2, 3, 5))
    oq = lqr._operand(Q, 2, (2, 3, 5))
    ox = lqr._operand(x0, 1, (2, 3, 5))
    assert list(oa.bstride) == [0, 16, 0] and oa.dtype == lqr.TTC_F32
    assert list(oq.bstride) == [240, 80, 16]
    assert list(ox.bstride) == [60, 20, 4] and ox.dtype == lqr.TTC_BF16
    with pytest.raises(ValueError):
        lqr._operand(Q.transpose(-1, -2), 2, (2, 3, 5))
    with pytest.raises(ValueError):
        lqr._operand(torch.zeros((4, 3, 5, 4, 4)), 2, (2, 3, 5))
    with pytest.raises(TypeError):
        lqr._operand(Q.double(), 2, (2, 3, 5))
