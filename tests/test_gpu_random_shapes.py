"""Seeded random geometries through the tensor-core kernel against the oracle, every element: filters of
1..5 x 1..5 taps (square or not), strides 1 and 2, the three padding modes, ragged channel counts, and
batches large enough that a CTA works through more tiles than its barrier rings have slots."""
import numpy as np
import pytest

import oracle
import paper_2011_09398_b200 as lce
from gpu_util import run_bconv

pytestmark = pytest.mark.gpu


def random_case(rng):
    while True:
        big = rng.integers(0, 3) == 0          # many tiles per CTA: the rings of four barriers wrap
        n = int(rng.integers(16, 65)) if big else int(rng.integers(1, 7))
        h, w = int(rng.integers(20, 66)), int(rng.integers(20, 66))
        if not big and rng.integers(0, 2):
            h, w = int(rng.integers(1, 20)), int(rng.integers(1, 20))
        kh = int(rng.integers(1, 6))
        kw = int(rng.choice([kh, rng.integers(1, 6)]))
        s = int(rng.integers(1, 3))
        pad = int(rng.choice([lce.PAD_VALID, lce.PAD_SAME_ONE, lce.PAD_SAME_ZERO]))
        cin = int(rng.choice([rng.integers(1, 70), rng.integers(1, 300), 32, 64, 128, 256]))
        cout = int(rng.choice([rng.integers(1, 130), rng.integers(1, 300), 32, 64, 128]))
        if big:
            cin, cout = int(rng.choice([32, 64, 96, 128])), int(rng.choice([32, 64, 128]))
        if pad == lce.PAD_VALID and (h < kh or w < kw):
            continue
        if n * (h // s + 1) * (w // s + 1) * cout * kh * kw * cin > 3e9:
            continue
        return n, h, w, cin, cout, kh, kw, s, pad


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_geometries_match_the_oracle(seed):
    rng = np.random.default_rng(seed)
    checked = 0
    while checked < 12:
        n, h, w, cin, cout, kh, kw, s, pad = random_case(rng)
        a = (2 * rng.integers(0, 2, size=(n, h, w, cin)) - 1).astype(np.int8)
        wt = (2 * rng.integers(0, 2, size=(cout, kh, kw, cin)) - 1).astype(np.int8)
        aw, ww = oracle.bitpack_pm1(a), oracle.bitpack_pm1(wt)
        kwargs = dict(in_c=cin, padding=pad, stride=(s, s))
        what = f"n={n} {h}x{w}x{cin}->{cout} k{kh}x{kw} s{s} pad={pad}"
        try:
            got = run_bconv(aw, ww, dict(kwargs, out_type=lce.OUT_INT32), kernel_choice=lce.KERNEL_TENSOR, packed=True)
        except lce.LceError as e:
            assert e.status == 2, what    # a shape the kernel does not cover (shared memory): said so, nothing ran
            continue
        acc = oracle.bconv2d_acc(a, wt, (s, s), pad)
        np.testing.assert_array_equal(got, acc, err_msg=what)
        thr = np.rint(np.sqrt(kh * kw * cin) * rng.standard_normal(cout)).astype(np.int32)
        got = run_bconv(aw, ww, dict(kwargs, out_type=lce.OUT_BITPACKED), thr=thr, kernel_choice=lce.KERNEL_TENSOR, packed=True)
        np.testing.assert_array_equal(got, oracle.transform_bits(acc, thr), err_msg=what)
        mult = rng.uniform(0.5, 1.5, cout).astype(np.float32)
        bias = (0.1 * rng.standard_normal(cout)).astype(np.float32)
        act = int(rng.integers(0, 2))
        got = run_bconv(aw, ww, dict(kwargs, out_type=lce.OUT_FLOAT32, activation=act), mult=mult, bias=bias,
                        kernel_choice=lce.KERNEL_TENSOR, packed=True)
        np.testing.assert_array_equal(got, oracle.transform_float(acc, mult, bias, act), err_msg=what)
        checked += 1
    assert lce.lce_device_status() == 0
