"""The allocation-free host entry point (for callers that cannot call cudaMalloc, so cannot hand
lce_bconv2d_host a workspace) must give exactly what lce_bconv2d_host gives, and both must give what
the CPU oracle computes from the definition.  Calls in a row on different inputs: each one runs on an
array that still holds the previous one's data.
This file sorts last on purpose, so that a run stopping at the first failure has already run
everything else."""
import numpy as np
import pytest
import torch

import lce_workloads as wl
import oracle
import paper_2011_09398_b200 as lce

pytestmark = pytest.mark.gpu


def host_case(spec, seed_index):
    t = wl.conv_tensors(1, seed_index + 1, spec)
    x = wl.activations(1, seed_index, (spec.batch, spec.in_h, spec.in_w, spec.in_c))
    desc = lce.make_desc(spec.batch, spec.in_h, spec.in_w, spec.in_c, spec.out_c, (spec.kernel,) * 2,
                         (spec.stride,) * 2, spec.padding, spec.out_type)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h = dict(
        desc=desc, a=pin(oracle.bitpack(x).view(np.int32)), w=pin(oracle.bitpack_pm1(t.w_pm1).view(np.int32)),
        mult=pin(t.multiplier) if spec.out_type == wl.OUT_FLOAT32 else None,
        bias=pin(t.bias) if spec.out_type == wl.OUT_FLOAT32 else None,
        thr=pin(t.thresholds) if spec.out_type == wl.OUT_BITPACKED else None)
    last = (spec.out_c + 31) // 32 if spec.out_type == wl.OUT_BITPACKED else spec.out_c
    dtype = torch.float32 if spec.out_type == wl.OUT_FLOAT32 else torch.int32
    shape = (spec.batch, spec.out_h, spec.out_w, last)
    acc = oracle.bconv2d_acc(oracle.sign(x), t.w_pm1, (spec.stride, spec.stride), spec.padding)
    if spec.out_type == wl.OUT_FLOAT32:
        ref = oracle.transform_float(acc, t.multiplier, t.bias)
    elif spec.out_type == wl.OUT_BITPACKED:
        ref = oracle.transform_bits(acc, t.thresholds).view(np.int32)
    else:
        ref = acc
    return h, shape, dtype, ref


def test_no_alloc_entry_point_matches_workspace_entry_point_twice_in_a_row():
    specs = [
        wl.ConvSpec("na_float", 2, 14, 14, 64, 64, 3, 1, wl.PAD_SAME_ONE, wl.OUT_FLOAT32),
        wl.ConvSpec("na_bits", 3, 9, 11, 40, 70, 3, 2, wl.PAD_SAME_ONE, wl.OUT_BITPACKED),
        wl.ConvSpec("na_int32", 2, 8, 8, 96, 33, 5, 1, wl.PAD_SAME_ZERO, wl.OUT_INT32),
    ]
    side_stream = torch.cuda.Stream(device="cuda:0")
    for k, spec in enumerate(specs):
        h, shape, dtype, ref = host_case(spec, 40 + 10 * k)
        assert lce.lce_bconv2d_host_workspace_bytes(h["desc"]) <= lce.lce_bconv2d_host_noalloc_max_bytes()
        want = torch.empty(shape, dtype=dtype).pin_memory()
        ws = torch.empty(lce.lce_bconv2d_host_workspace_bytes(h["desc"]), dtype=torch.uint8, device="cuda:0")
        lce.lce_bconv2d_host(h["desc"], h["a"], h["w"], h["mult"], h["bias"], h["thr"], want, ws)
        got = torch.full(shape, 7, dtype=dtype).pin_memory()
        if k == 1:  # once on a stream other than the default one
            with torch.cuda.stream(side_stream):
                lce.lce_bconv2d_host_noalloc(h["desc"], h["a"], h["w"], h["mult"], h["bias"], h["thr"], got)
        else:
            lce.lce_bconv2d_host_noalloc(h["desc"], h["a"], h["w"], h["mult"], h["bias"], h["thr"], got)
        assert torch.equal(got, want), f"{spec.name}: outputs differ"  # same kernel, same bits: exact
        assert np.array_equal(got.numpy(), ref), f"{spec.name}: differs from the oracle"


def test_no_alloc_entry_point_accepts_the_largest_call_that_fits_and_rejects_the_next():
    """Batch sizes on either side of the 8 MiB array for one layer shape (float 28x28x64 -> 64)."""
    limit = lce.lce_bconv2d_host_noalloc_max_bytes()
    mk = lambda n: lce.make_desc(n, 28, 28, 64, 64, out_type=lce.OUT_FLOAT32)
    n_fit = max(n for n in range(1, 200) if lce.lce_bconv2d_host_workspace_bytes(mk(n)) <= limit)
    spec = wl.ConvSpec("na_edge", n_fit, 28, 28, 64, 64, 3, 1, wl.PAD_SAME_ONE, wl.OUT_FLOAT32)
    h, shape, dtype, ref = host_case(spec, 90)
    got = torch.empty(shape, dtype=dtype).pin_memory()
    lce.lce_bconv2d_host_noalloc(h["desc"], h["a"], h["w"], h["mult"], h["bias"], h["thr"], got)
    assert np.array_equal(got.numpy(), ref)
    bigger = wl.ConvSpec("na_over", n_fit + 1, 28, 28, 64, 64, 3, 1, wl.PAD_SAME_ONE, wl.OUT_FLOAT32)
    h2, shape2, dtype2, _ = host_case(bigger, 91)
    with pytest.raises(lce.LceError) as e:
        lce.lce_bconv2d_host_noalloc(h2["desc"], h2["a"], h2["w"], h2["mult"], h2["bias"], h2["thr"], torch.empty(shape2, dtype=dtype2))
    assert e.value.status == 6


def test_no_alloc_entry_point_rejects_what_does_not_fit():
    spec = wl.ConvSpec("na_big", 64, 56, 56, 64, 64, 3, 1, wl.PAD_SAME_ONE, wl.OUT_FLOAT32)
    desc = lce.make_desc(spec.batch, spec.in_h, spec.in_w, spec.in_c, spec.out_c, out_type=lce.OUT_FLOAT32)
    assert lce.lce_bconv2d_host_workspace_bytes(desc) > lce.lce_bconv2d_host_noalloc_max_bytes()
    z = lambda n, dt: torch.zeros(n, dtype=dt)
    with pytest.raises(lce.LceError) as e:
        lce.lce_bconv2d_host_noalloc(desc, z(64 * 56 * 56 * 2, torch.int32), z(64 * 9 * 2, torch.int32), z(64, torch.float32),
                                     z(64, torch.float32), None, z(64 * 56 * 56 * 64, torch.float32))
    assert e.value.status == 6
