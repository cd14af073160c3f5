"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and rejects malformed calls before touching the device."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest

import paper_2011_09398_b200 as lce
from paper_2011_09398_b200 import build as lce_build

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    lce_build.build()
    return lce.library()


def declared_symbols(header):
    text = (ROOT / "include" / header).read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lce_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols("lce.h")
    assert {"lce_bitpack", "lce_bconv2d", "lce_bmaxpool", "lce_device_status_reset"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in lce.h but not exported"
    # the measurement-only companion library has a header of its own
    probe = ctypes.CDLL(str(lce_build.PROBE_LIB))
    probe_names = declared_symbols("lce_probe.h")
    assert probe_names == ["lce_probe_pipe", "lce_probe_stage"]
    for name in probe_names:
        assert hasattr(probe, name), f"{name} declared in lce_probe.h but not exported"
    assert not hasattr(lib, "lce_probe_pipe") and not hasattr(lib, "lce_probe_stage")
    assert {h.name for h in (ROOT / "include").glob("*.h")} == {"lce.h", "lce_probe.h"}


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


# ---- launch plans (host arithmetic only): the work split the kernels rely on ----------------------

def _plan(N, H, W, Cin, Cout, k, s, padding=None, kernel_choice=None, out_type=None, packed=0):
    d = lce.make_desc(N, H, W, Cin, Cout, (k, k), (s, s), lce.PAD_SAME_ONE if padding is None else padding,
                      lce.OUT_BITPACKED if out_type is None else out_type, lce.ACT_NONE,
                      lce.KERNEL_AUTO if kernel_choice is None else kernel_choice, packed)
    oh, ow = lce.lce_bconv2d_out_shape(d)
    return lce.lce_bconv2d_plan(d), N * oh * ow


PLAN_SHAPES = [(64, 56, 56, 64, 64, 3, 1), (64, 28, 28, 128, 128, 3, 1), (64, 14, 14, 256, 256, 3, 1), (64, 7, 7, 512, 512, 3, 1),
               (64, 56, 56, 64, 128, 3, 2), (1, 14, 14, 64, 64, 3, 1), (1, 8, 8, 32, 32, 3, 1), (64, 64, 64, 96, 96, 5, 1),
               (64, 64, 64, 256, 256, 5, 1), (3, 9, 11, 160, 70, 3, 1), (1, 1, 1, 33, 1, 3, 1), (2, 17, 13, 96, 33, 5, 2),
               (256, 112, 112, 32, 64, 3, 2), (7, 5, 5, 40, 200, 3, 1)]


@pytest.mark.parametrize("shape", PLAN_SHAPES)
def test_tiled_plan_covers_every_pixel_once_and_fits_the_sm(lib, shape):
    plan, M = _plan(*shape)
    Cout = shape[4]
    assert plan["kernel"] == lce.KERNEL_TILED and not plan["patch"] and not plan["pointwise"]
    nw, tp = plan["warps_per_cta"], plan["pixels_per_thread"]
    assert nw in (4, 8) and 1 <= tp <= 4 and (tp > 1 or nw == 4)
    assert plan["tile_pixels"] % (4 * nw * tp) == 0 and plan["tile_pixels"] > 0
    assert 0 < plan["shared_bytes"] <= 227 * 1024
    blocks = (Cout + 63) // 64
    half = plan["ctas_half_block"]
    full_blocks = blocks - (1 if half else 0)
    if half:
        assert 1 <= Cout % 64 <= 32
        r = plan["pixels_per_cta_half_block"]
        assert r % (8 * nw) == 0 and half * r >= M and (half - 1) * r < M   # ranges tile [0, M), none is empty
    if full_blocks:
        assert (plan["ctas"] - half) % full_blocks == 0
        per_block = (plan["ctas"] - half) // full_blocks
        r = plan["pixels_per_cta"]
        assert r % (4 * nw) == 0 and per_block * r >= M and (per_block - 1) * r < M
    # one resident wave: the kernel is persistent, no CTA waits for an SM
    per_sm_by_regs = (24 if tp <= 2 else 16) // nw
    per_sm_by_smem = (228 * 1024) // (plan["shared_bytes"] + 1024)
    assert plan["ctas"] <= 148 * min(per_sm_by_regs, per_sm_by_smem)


def test_plan_names_the_other_kernels(lib):
    assert _plan(2, 20, 18, 3, 32, 3, 2)[0]["patch"] == 1                                   # RGB stem: one-word patches
    p = _plan(64, 14, 14, 256, 512, 1, 1)[0]
    assert p["kernel"] == lce.KERNEL_TILED and p["pointwise"] == 1 and p["ctas"] > 0
    assert _plan(1, 9, 9, 64, 64, 7, 1)[0]["kernel"] == lce.KERNEL_DIRECT                    # no tiled 7x7
    assert _plan(1, 3, 4, 7300, 5, 3, 1)[0]["kernel"] == lce.KERNEL_DIRECT                   # K >= 65536 (and far more weights than shared memory holds)
    assert _plan(1, 9, 9, 64, 64, 3, 1, kernel_choice=lce.KERNEL_DIRECT)[0]["kernel"] == lce.KERNEL_DIRECT
    assert _plan(1, 9, 9, 64, 64, 3, 1, kernel_choice=lce.KERNEL_TENSOR, packed=1)[0]["kernel"] == lce.KERNEL_TENSOR
    with pytest.raises(lce.LceError) as e:
        _plan(1, 9, 9, 64, 64, 7, 1, kernel_choice=lce.KERNEL_TILED)
    assert e.value.status == 2
    with pytest.raises(lce.LceError) as e:
        _plan(1, 9, 9, 64, 64, 3, 1, kernel_choice=lce.KERNEL_TENSOR)                        # tensor path: packed weights only
    assert e.value.status == 2
    with pytest.raises(lce.LceError) as e:
        _plan(1, 9, 9, 64, 64, 3, 3, kernel_choice=lce.KERNEL_TENSOR, packed=1)              # tensor path: strides 1 and 2
    assert e.value.status == 2
    with pytest.raises(lce.LceError) as e:
        _plan(1, 9, 9, 1056, 64, 3, 1, kernel_choice=lce.KERNEL_TENSOR, packed=1)            # tensor path: at most 32 channel words
    assert e.value.status == 2


TENSOR_PLAN_SHAPES = [(64, 56, 56, 64, 64, 3, 1), (64, 28, 28, 128, 128, 3, 1), (64, 14, 14, 256, 256, 3, 1), (64, 7, 7, 512, 512, 3, 1),
                      (64, 56, 56, 64, 128, 3, 2), (64, 28, 28, 256, 256, 3, 2), (64, 14, 14, 256, 512, 1, 1), (256, 112, 112, 32, 64, 3, 2),
                      (64, 64, 64, 256, 256, 5, 1), (64, 32, 32, 96, 96, 5, 1), (128, 28, 28, 64, 128, 1, 1), (8, 9, 9, 512, 40, 7, 2)]


@pytest.mark.parametrize("out_type", [lce.OUT_BITPACKED, lce.OUT_FLOAT32])
@pytest.mark.parametrize("shape", TENSOR_PLAN_SHAPES)
def test_tensor_plan_fits_the_sm_and_auto_takes_it_for_large_packed_layers(lib, shape, out_type):
    forced, _ = _plan(*shape, kernel_choice=lce.KERNEL_TENSOR, out_type=out_type, packed=1)
    assert forced["kernel"] == lce.KERNEL_TENSOR
    assert forced["tile_pixels"] % 16 == 0 and 16 <= forced["tile_pixels"] <= 224       # N of the MMA, two accumulators in 512 columns
    assert 0 < forced["shared_bytes"] <= 227 * 1024
    assert 1 <= forced["ctas"] <= 148
    k = shape[5]
    assert min(2, k * k) <= forced["weight_stages"] <= k * k and forced["weights_resident"] == (forced["weight_stages"] == k * k)
    auto, M = _plan(*shape, out_type=out_type, packed=1)
    macs = M * shape[4] * k * k * shape[3]
    few_channels = shape[3] <= 32 and k * k <= 9
    threshold = 2 ** 31 if few_channels else 2 ** 28 if forced["weights_resident"] else 2 ** 29
    assert (auto["kernel"] == lce.KERNEL_TENSOR) == (macs >= threshold)
    assert _plan(*shape, out_type=out_type)[0]["kernel"] != lce.KERNEL_TENSOR             # plain weights: integer kernels


def test_packed_weights_buffer_holds_the_three_parts(lib):
    d = lce.make_desc(64, 28, 28, 128, 128, (3, 3), (1, 1))
    plain = 128 * 9 * 4 * 4
    total = lce.lce_bconv2d_packed_weights_bytes(d)
    tensor_image = 1 * 9 * 4 * 2048        # [channel block][tap][channel word][128 channels][16 bytes]
    assert total > plain + tensor_image and total % 256 == 0
    odd = lce.make_desc(1, 8, 8, 96, 130, (3, 3), (1, 1))   # 3 channel words are padded to 4, 130 channels to 2 blocks
    assert lce.lce_bconv2d_packed_weights_bytes(odd) >= 130 * 9 * 3 * 4 + 2 * 9 * 4 * 2048


def test_plans_are_remembered_per_geometry_not_mixed_up(lib):
    """The library keeps the last few plans of a host thread: a repeated geometry must give the same
    plan as the first time, with more distinct geometries in between than it keeps."""
    rng = np.random.default_rng(5)
    shapes = list(PLAN_SHAPES)
    for _ in range(30):
        k = int(rng.choice([1, 3, 5]))
        shapes.append((int(rng.integers(1, 9)), int(rng.integers(5, 40)), int(rng.integers(5, 40)), int(rng.integers(1, 200)),
                       int(rng.integers(1, 200)), k, int(rng.integers(1, 3))))
    first = [_plan(*s)[0] for s in shapes]
    again = [_plan(*s)[0] for s in reversed(shapes)][::-1]
    assert first == again
    # a field that is not part of the tile choice but is part of the geometry: output type and padding
    a = _plan(4, 20, 20, 64, 96, 3, 1, out_type=lce.OUT_FLOAT32)[0]
    b = _plan(4, 20, 20, 64, 96, 3, 1, padding=lce.PAD_VALID)[0]
    c = _plan(4, 20, 20, 64, 96, 3, 1, out_type=lce.OUT_FLOAT32)[0]
    assert a == c and b["kernel"] == lce.KERNEL_TILED


def test_plan_objects_check_their_arguments_on_the_host(lib):
    d = lce.make_desc(1, 4, 4, 32, 32)
    fake = ctypes.c_void_p(256)  # never dereferenced: nothing is launched by plan_create
    handle = ctypes.c_void_p()
    assert lib.lce_bconv2d_plan_create(ctypes.byref(d), None, fake, fake, fake, None, fake, ctypes.byref(handle)) == 1
    assert handle.value is None
    assert lib.lce_bconv2d_plan_create(ctypes.byref(d), fake, fake, fake, fake, None, fake, None) == 1      # nowhere to put the handle
    assert lib.lce_bconv2d_plan_create(ctypes.byref(d), ctypes.c_void_p(258), fake, fake, fake, None, fake, ctypes.byref(handle)) == 3
    forced = lce.make_desc(1, 9, 9, 64, 64, (3, 3), (2, 2), kernel_choice=lce.KERNEL_TENSOR)                   # tensor path: packed weights only
    assert lib.lce_bconv2d_plan_create(ctypes.byref(forced), fake, fake, fake, fake, None, fake, ctypes.byref(handle)) == 2
    assert lib.lce_bconv2d_plan_create(ctypes.byref(d), fake, fake, fake, fake, None, fake, ctypes.byref(handle)) == 0
    assert handle.value
    lib.lce_plan_destroy(handle)
    lib.lce_plan_destroy(None)                                                                                # ignored
    assert lib.lce_plan_run(None, None) == 1
