import ctypes
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
# the library honours its RESQ_* debugging overrides (which the tests use to reach every kernel variant) only when
# this is set before its first call
os.environ.setdefault("RESQ_DEBUG", "1")
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def nvref():
    """NVIDIA's host-callable fp4 / e8m0 conversions (toolkit headers), used as library pins."""
    src = os.path.join(ROOT, "tests", "helpers", "nv_cvt_ref.cpp")
    out = os.path.join(ROOT, "tests", "helpers", "libnv_cvt_ref.so")
    inc = "/usr/local/cuda/include"
    if not os.path.exists(os.path.join(inc, "cuda_fp4.h")):
        pytest.skip("CUDA toolkit headers not found")
    if not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        subprocess.check_call(["g++", "-O1", "-shared", "-fPIC", "-I" + inc, src, "-o", out])
    L = ctypes.CDLL(out)
    L.nv_float_to_e2m1.argtypes = [ctypes.c_float]
    L.nv_float_to_e2m1.restype = ctypes.c_int
    L.nv_e2m1_to_float.argtypes = [ctypes.c_int]
    L.nv_e2m1_to_float.restype = ctypes.c_float
    L.nv_e8m0_to_float.argtypes = [ctypes.c_int]
    L.nv_e8m0_to_float.restype = ctypes.c_float
    return L
