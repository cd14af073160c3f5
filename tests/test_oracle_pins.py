"""Pins for the CPU oracle: each test checks oracle/ against something other than
itself -- a fact the paper prints, a closed form, a library routine used by its
textbook meaning (torch's float convolution / max-pool, numpy's matrix product),
Python big-integer popcounts, or brute force in pure Python on tiny inputs.
None of these needs a GPU."""
import itertools
import math
from pathlib import Path

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from oracle import PAD_SAME_ONE, PAD_SAME_ZERO, PAD_VALID

GOLDEN = Path(__file__).parent / "golden" / "paper_facts.txt"


def golden():
    facts = {}
    for line in GOLDEN.read_text().splitlines():
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            facts[k.strip()] = v.strip()
    return facts


def rand_pm1(rng, shape):
    return (2 * rng.integers(0, 2, size=shape) - 1).astype(np.int8)


def tf_same_pads(size, k, s):
    out = -(-size // s)
    total = max((out - 1) * s + k - size, 0)
    return total // 2, total - total // 2


def torch_conv_acc(a, w, stride, padding):
    """Independent route: float convolution of the +-1 tensors with explicit padding.
    Exact in fp32 because every partial sum is an integer far below 2**24."""
    x = torch.from_numpy(a.astype(np.float32)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(w.astype(np.float32)).permute(0, 3, 1, 2)
    KH, KW = w.shape[1], w.shape[2]
    if padding != PAD_VALID:
        pt, pb = tf_same_pads(a.shape[1], KH, stride)
        pl, pr = tf_same_pads(a.shape[2], KW, stride)
        x = F.pad(x, (pl, pr, pt, pb), value=1.0 if padding == PAD_SAME_ONE else 0.0)
    y = F.conv2d(x.double(), wt.double(), stride=stride)
    return y.permute(0, 2, 3, 1).round().to(torch.int32).numpy()


FUZZ_SHAPES = [
    # N, H, W, Cin, Cout, k, s
    (1, 1, 1, 1, 1, 1, 1), (2, 5, 7, 3, 4, 3, 1), (1, 6, 6, 31, 5, 3, 2), (2, 7, 5, 32, 33, 3, 1),
    (1, 9, 8, 33, 31, 5, 1), (1, 8, 9, 64, 32, 5, 2), (3, 4, 4, 96, 64, 1, 1), (1, 7, 7, 40, 3, 1, 2),
    (1, 2, 3, 64, 2, 3, 1), (2, 14, 14, 64, 8, 3, 2), (1, 3, 3, 5, 7, 3, 1),
]


@pytest.mark.parametrize("padding", [PAD_VALID, PAD_SAME_ONE, PAD_SAME_ZERO])
@pytest.mark.parametrize("shape", FUZZ_SHAPES)
def test_acc_matches_float_convolution(shape, padding):
    N, H, W, Cin, Cout, k, s = shape
    if padding == PAD_VALID and (H < k or W < k):
        pytest.skip("empty VALID output")
    rng = np.random.default_rng(hash(shape) % 2**32)
    a, w = rand_pm1(rng, (N, H, W, Cin)), rand_pm1(rng, (Cout, k, k, Cin))
    got = oracle.bconv2d_acc(a, w, (s, s), padding)
    want = torch_conv_acc(a, w, s, padding)
    assert got.shape == want.shape
    np.testing.assert_array_equal(got, want)


def py_popcount(v):
    return bin(int(v)).count("1")


@pytest.mark.parametrize("shape", [(1, 4, 5, 3, 3, 3, 1), (2, 5, 4, 33, 4, 3, 2), (1, 3, 3, 64, 5, 1, 1), (1, 6, 6, 40, 2, 5, 1)])
def test_xor_popcount_and_and_popcount_identities(shape):
    """acc = K - 2*popc(a^w) and acc = K - 2popc(a) - 2popc(w) + 4popc(a&w) with Python
    big-int popcounts on the packed words; out-of-image taps read zero words (one-padding)."""
    N, H, W, Cin, Cout, k, s = shape
    rng = np.random.default_rng(7)
    a, w = rand_pm1(rng, (N, H, W, Cin)), rand_pm1(rng, (Cout, k, k, Cin))
    aw, ww = oracle.bitpack_pm1(a), oracle.bitpack_pm1(w)
    acc = oracle.bconv2d_acc(a, w, (s, s), PAD_SAME_ONE)
    _, OH, OW, _ = acc.shape
    pt, _ = tf_same_pads(H, k, s)
    pl, _ = tf_same_pads(W, k, s)
    K = k * k * Cin
    nw = aw.shape[-1]
    for n, oh, ow, o in itertools.product(range(N), range(OH), range(OW), range(Cout)):
        x = pa = pw = pand = 0
        for ky, kx, j in itertools.product(range(k), range(k), range(nw)):
            iy, ix = oh * s - pt + ky, ow * s - pl + kx
            av = int(aw[n, iy, ix, j]) if 0 <= iy < H and 0 <= ix < W else 0
            wv = int(ww[o, ky, kx, j])
            x += py_popcount(av ^ wv)
            pa += py_popcount(av); pw += py_popcount(wv); pand += py_popcount(av & wv)
        assert acc[n, oh, ow, o] == K - 2 * x
        assert acc[n, oh, ow, o] == K - 2 * pa - 2 * pw + 4 * pand


def test_brute_force_pure_python_tiny():
    rng = np.random.default_rng(11)
    N, H, W, Cin, Cout, k, s = 1, 4, 3, 5, 2, 3, 2
    a, w = rand_pm1(rng, (N, H, W, Cin)), rand_pm1(rng, (Cout, k, k, Cin))
    for padding, padval in ((PAD_SAME_ONE, 1), (PAD_SAME_ZERO, 0)):
        acc = oracle.bconv2d_acc(a, w, (s, s), padding)
        OH, OW = -(-H // s), -(-W // s)
        pt, pl = tf_same_pads(H, k, s)[0], tf_same_pads(W, k, s)[0]
        for oh, ow, o in itertools.product(range(OH), range(OW), range(Cout)):
            tot = 0
            for ky, kx, c in itertools.product(range(k), range(k), range(Cin)):
                iy, ix = oh * s - pt + ky, ow * s - pl + kx
                v = int(a[0, iy, ix, c]) if 0 <= iy < H and 0 <= ix < W else padval
                tot += v * int(w[o, ky, kx, c])
            assert acc[0, oh, ow, o] == tot


def test_flipping_weights_negates_accumulator():
    rng = np.random.default_rng(3)
    a, w = rand_pm1(rng, (2, 6, 5, 37)), rand_pm1(rng, (6, 3, 3, 37))
    for padding in (PAD_VALID, PAD_SAME_ONE, PAD_SAME_ZERO):
        np.testing.assert_array_equal(oracle.bconv2d_acc(a, -w, (1, 1), padding),
                                      -oracle.bconv2d_acc(a, w, (1, 1), padding))


def test_pointwise_conv_is_matrix_product():
    rng = np.random.default_rng(4)
    a, w = rand_pm1(rng, (2, 3, 4, 70)), rand_pm1(rng, (9, 1, 1, 70))
    acc = oracle.bconv2d_acc(a, w, (1, 1), PAD_SAME_ONE)
    want = a.reshape(-1, 70).astype(np.int64) @ w.reshape(9, 70).astype(np.int64).T
    np.testing.assert_array_equal(acc.reshape(-1, 9), want)


def test_parity_and_range_invariants():
    rng = np.random.default_rng(5)
    a, w = rand_pm1(rng, (1, 5, 5, 35)), rand_pm1(rng, (4, 3, 3, 35))
    K = 9 * 35
    acc = oracle.bconv2d_acc(a, w, (1, 1), PAD_SAME_ONE)
    assert np.all((acc - K) % 2 == 0) and np.all(np.abs(acc) <= K)


@pytest.mark.parametrize("Cin", [1, 32, 40])
def test_one_padding_closed_forms(Cin):
    H = W = 5
    K = 9 * Cin
    ones = np.ones((1, H, W, Cin), np.int8)
    wpos = np.ones((3, 3, 3, Cin), np.int8)
    # all +1 input and weights: K everywhere, borders included (padding is +1 too)
    assert np.all(oracle.bconv2d_acc(ones, wpos, (1, 1), PAD_SAME_ONE) == K)
    # all -1 input, +1 weights: the +1 padding shows at edges (3 taps) and corners (5 taps)
    acc = oracle.bconv2d_acc(-ones, wpos, (1, 1), PAD_SAME_ONE)[0, :, :, 0]
    assert np.all(acc[1:-1, 1:-1] == -K)
    assert acc[0, 2] == -K + 2 * 3 * Cin and acc[2, 0] == -K + 2 * 3 * Cin
    assert acc[0, 0] == -K + 2 * 5 * Cin and acc[-1, -1] == -K + 2 * 5 * Cin
    # zero padding, all +1: count of in-image taps
    accz = oracle.bconv2d_acc(ones, wpos, (1, 1), PAD_SAME_ZERO)[0, :, :, 0]
    assert accz[0, 0] == 4 * Cin and accz[0, 2] == 6 * Cin and accz[2, 2] == 9 * Cin


def test_same_geometry_shapes_and_asymmetric_pad():
    for size, k, s, want in ((224, 3, 2, 112), (56, 3, 2, 28), (7, 3, 1, 7), (14, 1, 1, 14), (15, 3, 2, 8), (8, 5, 1, 8)):
        assert oracle.out_size(size, k, s, PAD_SAME_ONE) == want
    assert oracle.out_size(7, 3, 2, PAD_VALID) == 3 and oracle.out_size(2, 3, 1, PAD_VALID) == 0
    # TensorFlow SAME, 3x3 stride 2 on an even size: no pad before, one after
    assert oracle.pad_before(56, 3, 2, PAD_SAME_ONE) == 0
    assert oracle.pad_before(56, 3, 1, PAD_SAME_ONE) == 1
    assert oracle.pad_before(15, 3, 2, PAD_SAME_ONE) == 1
    assert oracle.pad_before(8, 5, 1, PAD_SAME_ONE) == 2 and oracle.pad_before(9, 1, 2, PAD_SAME_ONE) == 0
    # a single -1 row at the bottom of a 4x4 input: with pad (0 before, 1 after) the last
    # output row (input rows 2,3,pad) sees it, the first (rows 0,1,2) does not.
    a = np.ones((1, 4, 4, 1), np.int8)
    a[0, 3] = -1
    w = np.ones((1, 3, 3, 1), np.int8)
    acc = oracle.bconv2d_acc(a, w, (2, 2), PAD_SAME_ONE)[0, :, :, 0]
    assert acc.shape == (2, 2)
    assert acc[0, 0] == 9          # rows 0..2, cols 0..2: all +1
    assert acc[1, 0] == 9 - 2 * 3  # rows 2,3,pad: three -1 taps (cols 0..2 of row 3)
    assert acc[1, 1] == 9 - 2 * 2  # cols 2,3,pad: two -1 taps


def test_bit_convention_and_sizes_from_the_paper():
    g = golden()
    x = np.array([[1.5, -2.0, 0.0, -0.0, float("nan"), -1e-30, 3.0]], np.float32)
    words = oracle.bitpack(x)
    bits = [(int(words[0, 0]) >> i) & 1 for i in range(7)]
    plus, minus = int(g["bit_for_plus_one"]), int(g["bit_for_minus_one"])
    assert bits == [plus, minus, plus, plus, plus, minus, plus]
    # channels padded up to a multiple of 32; pad bits are zero
    mult = int(g["channel_pad_multiple"])
    for C in (1, 3, 31, 32, 33, 64, 65):
        w = oracle.bitpack(-np.ones((2, C), np.float32))
        assert w.shape == (2, -(-C // mult)) and w.dtype == np.uint32
        assert sum(py_popcount(v) for v in w[0]) == C
    # 32x smaller than float, 8x smaller than 8-bit
    xf = np.zeros((3, 4, 4, 64), np.float32)
    assert xf.nbytes == int(g["packed_vs_float_ratio"]) * oracle.bitpack(xf).nbytes
    assert xf.astype(np.int8).nbytes == int(g["packed_vs_int8_ratio"]) * oracle.bitpack(xf).nbytes
    # 256 filters of 3x3 on 256 channels = 72 KiB packed
    wts = oracle.bitpack_pm1(np.ones((256, 3, 3, 256), np.int8))
    assert wts.nbytes == int(g["weights_256x3x3x256_kib"]) * 1024


def test_bit_order_one_hot():
    # reading: channel c -> word c//32, bit c%32 (LSB = lowest channel)
    for C, c in ((70, 0), (70, 31), (70, 32), (70, 69)):
        x = np.ones((1, C), np.float32)
        x[0, c] = -1.0
        w = oracle.bitpack(x)
        assert int(w[0, c // 32]) == 1 << (c % 32)
        assert sum(int(v != 0) for v in w[0]) == 1


def test_unpack_inverts_bitpack():
    rng = np.random.default_rng(8)
    x = rng.standard_normal((5, 3, 77)).astype(np.float32)
    x[0, 0, :4] = [0.0, -0.0, np.nan, -np.inf]
    want = np.where(x < 0, -1, 1).astype(np.int8)
    np.testing.assert_array_equal(oracle.unpack_pm1(oracle.bitpack(x), 77), want)
    np.testing.assert_array_equal(oracle.unpack_f32(oracle.bitpack(x), 77), want.astype(np.float32))
    np.testing.assert_array_equal(oracle.sign(x), want)
    np.testing.assert_array_equal(oracle.bitpack_pm1(want), oracle.bitpack(x))


@pytest.mark.parametrize("pool,stride,padding", [((2, 2), (2, 2), PAD_VALID), ((3, 3), (2, 2), PAD_SAME_ONE), ((2, 3), (1, 2), PAD_VALID), ((3, 3), (1, 1), PAD_SAME_ONE)])
def test_bmaxpool_is_sign_of_float_maxpool(pool, stride, padding):
    """max(sign X) = sign(max X) (Section 3.2, LceBMaxPool2d) against torch's float max-pool;
    would fail if the bit polarity were the other way round."""
    rng = np.random.default_rng(9)
    N, H, W, C = 2, 7, 9, 45
    x = rng.standard_normal((N, H, W, C)).astype(np.float32)
    xt = torch.from_numpy(x).permute(0, 3, 1, 2)
    if padding != PAD_VALID:
        pt, pb = tf_same_pads(H, pool[0], stride[0])
        pl, pr = tf_same_pads(W, pool[1], stride[1])
        xt = F.pad(xt, (pl, pr, pt, pb), value=-float("inf"))
    pooled = F.max_pool2d(xt, pool, stride).permute(0, 2, 3, 1).numpy()
    got = oracle.bmaxpool(oracle.bitpack(x), C, pool, stride, padding)
    np.testing.assert_array_equal(got, oracle.bitpack(pooled))
    # and it is the bitwise AND of the window's words (VALID 2x2 case spelled out)
    if pool == (2, 2) and padding == PAD_VALID:
        w = oracle.bitpack(x)
        want = w[:, 0:6:2, 0:8:2] & w[:, 1:7:2, 0:8:2] & w[:, 0:6:2, 1:9:2] & w[:, 1:7:2, 1:9:2]
        np.testing.assert_array_equal(got, want)


def test_float_transform_closed_form():
    rng = np.random.default_rng(10)
    acc = rng.integers(-4608, 4609, size=(50, 9)).astype(np.int32)
    m = rng.uniform(0.5, 1.5, 9).astype(np.float32)
    b = (0.1 * rng.standard_normal(9)).astype(np.float32)
    # one rounding: the exact product+sum in double (53 bits hold 24x24-bit products + add
    # exactly enough here to round once), then a single cast
    want = (acc.astype(np.float64) * m.astype(np.float64) + b.astype(np.float64)).astype(np.float32)
    np.testing.assert_array_equal(oracle.transform_float(acc, m, b), want)
    relu = np.maximum(acc, 0)
    want_relu = (relu.astype(np.float64) * m.astype(np.float64) + b.astype(np.float64)).astype(np.float32)
    np.testing.assert_array_equal(oracle.transform_float(acc, m, b, oracle.ACT_RELU), want_relu)
    one, zero = np.ones(9, np.float32), np.zeros(9, np.float32)
    np.testing.assert_array_equal(oracle.transform_float(acc, one, zero), acc.astype(np.float32))


def test_threshold_equals_sign_of_float_output():
    """Bit-packed output == LceQuantize of the float output when thr = ceil(-bias/mult), mult > 0
    (the converter's fusion, Section 3.1); plus the two saturated thresholds."""
    rng = np.random.default_rng(12)
    a, w = rand_pm1(rng, (2, 6, 6, 64)), rand_pm1(rng, (40, 3, 3, 64))
    acc = oracle.bconv2d_acc(a, w, (1, 1), PAD_SAME_ONE)
    m = rng.uniform(0.5, 1.5, 40).astype(np.float32)
    cut = rng.integers(-60, 60, size=40) + 0.5           # never an integer
    b = (-cut * m.astype(np.float64)).astype(np.float32)
    ratio = -b.astype(np.float64) / m.astype(np.float64)
    assert np.all(np.abs(ratio - np.rint(ratio)) > 0.1)
    thr = np.ceil(ratio).astype(np.int32)
    fl = oracle.transform_float(acc, m, b)
    np.testing.assert_array_equal(oracle.transform_bits(acc, thr), oracle.bitpack(fl))
    lo = np.full(40, np.iinfo(np.int32).min, np.int32)
    hi = np.full(40, np.iinfo(np.int32).max, np.int32)
    assert not oracle.transform_bits(acc, lo).any()
    allones = oracle.transform_bits(acc, hi)
    assert np.all(allones[..., 0] == 0xFFFFFFFF) and np.all(allones[..., 1] == 0xFF)  # 40 channels: pad bits 0


def test_sampled_outputs_match_full():
    rng = np.random.default_rng(13)
    a, w = rand_pm1(rng, (3, 9, 8, 33)), rand_pm1(rng, (7, 3, 3, 33))
    for s, padding in ((1, PAD_SAME_ONE), (2, PAD_SAME_ONE), (2, PAD_SAME_ZERO), (1, PAD_VALID)):
        acc = oracle.bconv2d_acc(a, w, (s, s), padding)
        idx = np.stack([rng.integers(0, d, size=64) for d in acc.shape], axis=1).astype(np.int32)
        got = oracle.bconv2d_acc_at(a, w, idx, (s, s), padding)
        np.testing.assert_array_equal(got, acc[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]])


def test_add_is_one_fp32_rounding():
    rng = np.random.default_rng(14)
    a = rng.standard_normal(1000).astype(np.float32) * 1e3
    b = rng.standard_normal(1000).astype(np.float32)
    want = (a.astype(np.float64) + b.astype(np.float64)).astype(np.float32)
    np.testing.assert_array_equal(oracle.add_f32(a, b), want)


def test_bitpacked_chaining_equals_float_then_quantize():
    """A binarized layer feeding another may emit bits directly instead of float + LceQuantize
    (Section 3.2, LceQuantize, last sentence)."""
    rng = np.random.default_rng(15)
    a, w1, w2 = rand_pm1(rng, (1, 6, 6, 32)), rand_pm1(rng, (32, 3, 3, 32)), rand_pm1(rng, (8, 3, 3, 32))
    acc1 = oracle.bconv2d_acc(a, w1, (1, 1), PAD_SAME_ONE)
    m = np.ones(32, np.float32)
    b = np.full(32, 0.5, np.float32)
    direct = oracle.transform_bits(acc1, np.zeros(32, np.int32))       # acc < 0  <=>  acc + 0.5 < 0
    via_float = oracle.bitpack(oracle.transform_float(acc1, m, b))
    np.testing.assert_array_equal(direct, via_float)
    out_a = oracle.bconv2d_acc(oracle.unpack_pm1(direct, 32), w2, (1, 1), PAD_SAME_ONE)
    out_b = oracle.bconv2d_acc(oracle.sign(oracle.transform_float(acc1, m, b)), w2, (1, 1), PAD_SAME_ONE)
    np.testing.assert_array_equal(out_a, out_b)
