"""The measurement-only companion library on the GPU: the staging probe runs its three copy forms and
rejects what a 16-byte copy cannot do; the pipe probe reports a positive rate."""
import ctypes

import pytest
import torch

from paper_2011_09398_b200 import build as lce_build

pytestmark = pytest.mark.gpu

LCE_OK, LCE_ERR_INVALID_ARG, LCE_ERR_UNSUPPORTED = 0, 1, 2


@pytest.fixture(scope="module")
def probe_lib():
    lib = ctypes.CDLL(str(lce_build.PROBE_LIB))
    lib.lce_probe_stage.argtypes = [ctypes.c_int32] * 7 + [ctypes.POINTER(ctypes.c_double)] * 2 + [ctypes.c_void_p]
    lib.lce_probe_stage.restype = ctypes.c_int
    lib.lce_probe_pipe.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
                                   ctypes.c_void_p]
    lib.lce_probe_pipe.restype = ctypes.c_int
    torch.zeros(1, device="cuda")
    return lib


def stage(lib, mode, batch, h, w, words, rows, passes=2):
    a, b = ctypes.c_double(-1.0), ctypes.c_double(-1.0)
    st = lib.lce_probe_stage(mode, batch, h, w, words, rows, passes, ctypes.byref(a), ctypes.byref(b), None)
    return st, a.value, b.value


@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("shape", [(8, 28, 28, 4, 7), (5, 7, 7, 16, 3), (3, 14, 14, 8, 14)])
def test_staging_probe_runs_every_copy_form(probe_lib, mode, shape):
    st, us, first = stage(probe_lib, mode, *shape)
    assert st == LCE_OK
    assert 0.0 < first < 1e4 and 0.0 < us < 1e5   # microseconds; no wait ran out (that would be status 5)


def test_staging_probe_rejects_what_it_cannot_copy(probe_lib):
    assert stage(probe_lib, 0, 4, 56, 56, 2, 4)[0] == LCE_OK            # 4-byte copies take any word count
    assert stage(probe_lib, 1, 4, 56, 56, 2, 4)[0] == LCE_ERR_UNSUPPORTED   # 8 contiguous bytes per pixel only
    assert stage(probe_lib, 2, 4, 56, 56, 2, 4)[0] == LCE_ERR_UNSUPPORTED
    assert stage(probe_lib, 3, 4, 28, 28, 4, 7)[0] == LCE_ERR_INVALID_ARG
    assert stage(probe_lib, 0, 4, 28, 28, 3, 7)[0] == LCE_ERR_INVALID_ARG   # word planes by shift and mask
    assert stage(probe_lib, 0, 0, 28, 28, 4, 7)[0] == LCE_ERR_INVALID_ARG


def test_pipe_probe_reports_a_rate(probe_lib):
    a, b = ctypes.c_double(), ctypes.c_double()
    assert probe_lib.lce_probe_pipe(3, 50, ctypes.byref(a), ctypes.byref(b), None) == LCE_OK
    assert a.value > 0 and b.value > 0
