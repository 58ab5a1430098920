"""Access to the TEST build of the library (csrc/testing.h): the CUDA-core cross-check kernel, the
kernel/split overrides and the wait-timeout probe.  Test infrastructure; the product never loads it."""
from __future__ import annotations

import contextlib
import ctypes

from paper_2505_20776_b200 import api, build

_TLIB = None


def load_testing_lib() -> ctypes.CDLL:
    global _TLIB
    if _TLIB is None:
        L = api.bind(build.build_testing())
        L.specext_test_set_tuning.restype = ctypes.c_int
        L.specext_test_set_tuning.argtypes = [ctypes.c_int32, ctypes.c_int32]
        L.specext_test_wait_timeout.restype = ctypes.c_int
        L.specext_test_wait_timeout.argtypes = [ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
        _TLIB = L
    return _TLIB


@contextlib.contextmanager
def tuned(attn_kernel: int = 0, min_tiles_per_cta: int = 0):
    """Inside the block the binding's calls go to the test library with the given overrides."""
    L = load_testing_lib()
    saved = api._LIB
    assert L.specext_test_set_tuning(attn_kernel, min_tiles_per_cta) == 0
    api._LIB = L
    try:
        yield L
    finally:
        L.specext_test_set_tuning(0, 1)
        api._LIB = saved
