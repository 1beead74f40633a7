"""The C-ABI boundary without a GPU: the library loads, exports every function include/stwq.h
declares, and rejects bad arguments on the host before touching a device."""
import ctypes as C
import os
import re

import pytest

import paper_2601_21238_b200 as pk
from paper_2601_21238_b200 import build as pkbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pkbuild.build()
    return pk.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "stwq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return re.findall(r"^\s*(?:const\s+)?[A-Za-z_][\w\s\*]*?\b(\w+)\s*\([^;{]*\)\s*;", text, flags=re.M)


def test_every_declared_function_is_exported(lib):
    names = _declared()
    assert {"stwq_create", "stwq_destroy", "stwq_calibrate", "gps_fold", "stwq_quantize", "qlinear",
            "qlinear_q", "stwq_device_status", "stwq_strerror"} <= set(names)
    for n in names:
        assert getattr(lib, n) is not None
    assert set(pk.exported_symbols()) <= set(names)


def test_host_side_argument_errors(lib):
    # no context -> NULL error, before any CUDA call
    assert lib.qlinear(None, None, None, 1, 16, 16, None, None, None, 1, None, None, 8, 0, 0, None, None) == -1
    assert lib.stwq_quantize(None, None, None, 1, 16, None, None, 1, 8, None, None) == -1
    assert lib.gps_fold(None, None, 1, 1, None, 8, None, None, None) == -1
    assert lib.gps_scales(None, None, 1, 1, None, 1, 8, 999900, 0, None, None, None) == -1
    assert lib.stwq_calibrate(None, None, None, 1, 1, 1, None, 8, 1000000, None, None) == -1
    assert lib.stwq_strerror(0) == b"ok"
    assert b"NULL" in lib.stwq_strerror(-1)
    assert lib.stwq_strerror(-7) and lib.stwq_strerror(-123) == b"unknown status"
    h = C.c_void_p()
    rc = lib.stwq_create(C.byref(h), 0)
    import torch
    if not torch.cuda.is_available():
        assert rc != 0 and not h.value          # no device here: creation must fail, not fall back


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        pk.Context(0)
