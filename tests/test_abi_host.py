"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and rejects malformed calls before touching the device."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_2011_09398_b200 as lce
from paper_2011_09398_b200 import build as lce_build

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    lce_build.build()
    return lce.library()


def declared_symbols():
    text = (ROOT / "include" / "lce.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lce_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"lce_bitpack", "lce_bconv2d", "lce_bmaxpool"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in lce.h but not exported"


def test_version_and_status_strings(lib):
    assert "sm_100a" in lce.lce_version()
    assert lce.lce_status_string(0) == "ok"
    assert len({lce.lce_status_string(i) for i in range(7)}) == 7


def test_out_shape_follows_tensorflow_rules(lib):
    d = lce.make_desc(1, 224, 224, 3, 32, (3, 3), (2, 2), lce.PAD_SAME_ONE)
    assert lce.lce_bconv2d_out_shape(d) == (112, 112)
    d = lce.make_desc(1, 7, 7, 512, 512, (3, 3), (1, 1), lce.PAD_SAME_ONE)
    assert lce.lce_bconv2d_out_shape(d) == (7, 7)
    d = lce.make_desc(1, 7, 9, 8, 8, (3, 3), (2, 2), lce.PAD_VALID)
    assert lce.lce_bconv2d_out_shape(d) == (3, 4)
    with pytest.raises(lce.LceError) as e:
        lce.lce_bconv2d_out_shape(lce.make_desc(1, 2, 2, 8, 8, (3, 3), (1, 1), lce.PAD_VALID))  # empty output
    assert e.value.status == 1


def test_argument_errors_come_back_as_status_codes(lib):
    d = lce.make_desc(1, 4, 4, 32, 32)
    null = None
    fake = ctypes.c_void_p(256)  # never dereferenced: the checks below fail first
    assert lib.lce_bconv2d(ctypes.byref(d), null, fake, fake, fake, null, fake, null) == 1
    assert lib.lce_bconv2d(ctypes.byref(d), fake, fake, null, fake, null, fake, null) == 1      # float output needs multiplier
    d2 = lce.make_desc(1, 4, 4, 32, 32, out_type=lce.OUT_BITPACKED)
    assert lib.lce_bconv2d(ctypes.byref(d2), fake, fake, null, null, null, fake, null) == 1     # needs thresholds
    d3 = lce.make_desc(1, 4, 4, 32, 32, out_type=lce.OUT_BITPACKED, activation=lce.ACT_RELU)
    assert lib.lce_bconv2d(ctypes.byref(d3), fake, fake, null, null, fake, fake, null) == 1     # activation folded into thresholds
    bad = lce.make_desc(1, 4, 4, 32, 32, stride=(0, 1))
    assert lib.lce_bconv2d(ctypes.byref(bad), fake, fake, fake, fake, null, fake, null) == 1
    odd = ctypes.c_void_p(258)
    assert lib.lce_bconv2d(ctypes.byref(d), odd, fake, fake, fake, null, fake, null) == 3       # misaligned
    assert lib.lce_bitpack(null, fake, 4, 32, null) == 1
    assert lib.lce_bitpack(fake, fake, -1, 32, null) == 1
    assert lib.lce_bitpack(fake, fake, 0, 32, null) == 0                                       # empty input: no-op
    assert lib.lce_bitpack(fake, fake, 4, 0, null) == 1
    assert lib.lce_bmaxpool(fake, fake, 1, 4, 4, 32, 2, 2, 2, 2, lce.PAD_SAME_ZERO, null) == 1
    assert lib.lce_bmaxpool(fake, fake, 1, 1, 1, 32, 2, 2, 2, 2, lce.PAD_VALID, null) == 1      # empty output
    assert lib.lce_add_f32(fake, fake, fake, 0, null) == 0
    assert lib.lce_add_f32(null, fake, fake, 4, null) == 1
    assert lib.lce_bconv2d_host_workspace_bytes(ctypes.byref(bad)) == 0
    assert lib.lce_bconv2d_host_workspace_bytes(ctypes.byref(d)) >= 4 * 4 * 4 + 32 * 9 * 4 + 4 * 4 * 32 * 4


def test_binding_refuses_cpu_tensors():
    import torch
    with pytest.raises(ValueError):
        lce.lce_bitpack(torch.zeros(4, 32))
