"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Integer and bit outputs must be identical; float outputs must agree within
1e-6 * (|acc*multiplier| + |bias|) (the transform is a single fp32 multiply-add; the goal is 0 ulp)."""
import numpy as np
import pytest
import torch

import lce_workloads as wl
import oracle
import paper_2011_09398_b200 as lce
from gpu_util import DEV, guarded, guards_intact, run_bconv, to_dev, to_dev_words, words_to_host

pytestmark = pytest.mark.gpu

# (kernel choice, weights packed at load time?)
KERNELS = [(lce.KERNEL_DIRECT, False), (lce.KERNEL_AUTO, False), (lce.KERNEL_AUTO, True), (lce.KERNEL_TENSOR, True)]
KERNEL_IDS = ["direct", "auto", "auto-packed", "tensor"]


def skip_unless_covered(kernel_choice, N, H, W, Cin, Cout, k, s, padding):
    """The tensor-core kernel is forced in these tests; shapes it does not cover are reported as such."""
    if kernel_choice[0] != lce.KERNEL_TENSOR:
        return
    desc = lce.make_desc(N, H, W, Cin, Cout, (k, k), (s, s), padding, lce.OUT_FLOAT32, lce.ACT_NONE, lce.KERNEL_TENSOR, 1)
    try:
        lce.lce_bconv2d_plan(desc)
    except lce.LceError as e:
        assert e.status == 2
        pytest.skip("not covered by the tensor-core kernel")


def rand_pm1(rng, shape):
    return (2 * rng.integers(0, 2, size=shape) - 1).astype(np.int8)


def float_close(got, acc, mult, bias, act=0):
    v = np.maximum(acc, 0) if act else acc
    want = oracle.transform_float(acc, mult, bias, act)
    tol = 1e-6 * (np.abs(v.astype(np.float64) * mult.astype(np.float64)) + np.abs(bias.astype(np.float64)))
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    assert np.all(err <= tol), f"max err {err.max()}"
    return int((got != want).sum())


# ---- LceQuantize / LceDequantize ---------------------------------------------------------

@pytest.mark.parametrize("rows,C", [(1, 1), (7, 3), (50, 31), (33, 32), (129, 33), (1000, 40), (4097, 64), (300, 96),
                                    (513, 256), (2, 4096), (100003, 3), (4099, 1), (1026, 2), (8, 4), (5001, 4), (3, 3)])
def test_bitpack_matches_oracle(rows, C):
    rng = np.random.default_rng(rows * 131 + C)
    x = rng.standard_normal((rows, C)).astype(np.float32)
    x.flat[:6] = [0.0, -0.0, np.nan, -np.nan, np.inf, -np.inf][: min(6, x.size)]
    whole, out = guarded((rows, (C + 31) // 32), torch.int32, 0x5A5A5A5A)
    lce.lce_bitpack(to_dev(x), out)
    torch.cuda.synchronize()
    assert guards_intact(whole, 0x5A5A5A5A)
    np.testing.assert_array_equal(words_to_host(out), oracle.bitpack(x))


def test_bitpack_few_channels_from_an_unaligned_pointer():
    # 16-byte alignment decides between the 128-bit few-channel kernel and the generic one
    rng = np.random.default_rng(5)
    x = rng.standard_normal((1001, 3)).astype(np.float32)
    buf = torch.zeros(1001 * 3 + 1, dtype=torch.float32, device=DEV)
    buf[1:] = to_dev(x).flatten()
    got = words_to_host(lce.lce_bitpack(buf[1:].view(1001, 3)))
    np.testing.assert_array_equal(got, oracle.bitpack(x))


def test_bitpack_one_hot_bit_order():
    for C, c in ((64, 0), (64, 31), (64, 32), (70, 69)):
        x = np.ones((3, C), np.float32)
        x[1, c] = -1.0
        got = words_to_host(lce.lce_bitpack(to_dev(x)))
        np.testing.assert_array_equal(got, oracle.bitpack(x))
        assert int(got[1, c // 32]) == 1 << (c % 32)


@pytest.mark.parametrize("rows,C", [(5, 3), (64, 64), (77, 70), (1, 1), (4099, 32), (1001, 256), (3, 96)])
def test_unpack_matches_oracle(rows, C):
    rng = np.random.default_rng(C)
    words = oracle.bitpack(rng.standard_normal((rows, C)).astype(np.float32))
    got = lce.lce_unpack(to_dev_words(words), C).cpu().numpy()
    np.testing.assert_array_equal(got, oracle.unpack_f32(words, C))


def test_empty_bitpack_is_a_noop():
    x = torch.empty((0, 64), dtype=torch.float32, device=DEV)
    assert lce.lce_bitpack(x).shape == (0, 2)


# ---- LceBConv2d: fuzz over small ragged shapes --------------------------------------------

FUZZ = [
    # N, H, W, Cin, Cout, k, s
    (1, 1, 1, 1, 1, 1, 1), (2, 5, 7, 3, 4, 3, 1), (1, 6, 6, 31, 5, 3, 2), (2, 7, 5, 32, 33, 3, 1),
    (1, 9, 8, 33, 31, 5, 1), (1, 8, 9, 64, 32, 5, 2), (3, 4, 4, 96, 64, 1, 1), (1, 7, 7, 40, 3, 1, 2),
    (1, 2, 3, 64, 2, 3, 1), (2, 14, 14, 64, 64, 3, 1), (2, 14, 14, 64, 8, 3, 2), (1, 3, 3, 5, 7, 3, 1),
    (3, 7, 7, 512, 64, 3, 1), (2, 9, 11, 160, 70, 3, 1), (1, 17, 13, 96, 96, 3, 2), (2, 8, 8, 128, 130, 3, 1),
    (1, 29, 31, 64, 64, 3, 1), (2, 16, 16, 256, 32, 1, 1), (1, 57, 9, 32, 64, 3, 1), (5, 7, 7, 64, 64, 3, 1),
    # pointwise: channel words split into nine-word groups and leftover triples in every combination
    (1, 5, 5, 512, 70, 1, 1), (2, 6, 6, 200, 64, 1, 1), (1, 6, 5, 160, 8, 1, 1), (1, 4, 4, 320, 16, 1, 1),
    (2, 9, 9, 64, 128, 1, 2), (1, 28, 28, 128, 256, 1, 1), (1, 3, 5, 608, 33, 1, 1),
    # 5x5 filters: 25 taps = two full nine-word groups and one partial group per channel word
    (2, 16, 16, 64, 64, 5, 1), (1, 33, 29, 96, 70, 5, 1), (2, 17, 19, 160, 40, 5, 2), (3, 8, 8, 256, 256, 5, 1),
    (1, 4, 3, 32, 9, 5, 1), (1, 64, 64, 32, 32, 5, 1),
    # wide rows and 256 channels: weights too large for two CTAs per SM -> the eight-warp variant
    (1, 20, 64, 256, 70, 5, 1),
    # K = 9 * 7300 > 65535: past what the tiled kernel's 16-bit packed counts hold -> direct kernel
    (1, 3, 4, 7300, 5, 3, 1),
    # few input channels: the whole receptive field fits one word
    (2, 20, 18, 3, 32, 3, 2), (1, 9, 9, 1, 40, 5, 1), (1, 12, 11, 2, 70, 3, 1), (2, 8, 8, 3, 5, 3, 1),
]


@pytest.mark.parametrize("kernel_choice", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("padding", [lce.PAD_VALID, lce.PAD_SAME_ONE, lce.PAD_SAME_ZERO])
@pytest.mark.parametrize("shape", FUZZ)
def test_bconv_all_output_types_match_oracle(shape, padding, kernel_choice):
    N, H, W, Cin, Cout, k, s = shape
    if padding == lce.PAD_VALID and (H < k or W < k):
        pytest.skip("empty VALID output")
    skip_unless_covered(kernel_choice, N, H, W, Cin, Cout, k, s, padding)
    rng = np.random.default_rng(abs(hash((shape, padding))) % 2**32)
    a, w = rand_pm1(rng, (N, H, W, Cin)), rand_pm1(rng, (Cout, k, k, Cin))
    aw, ww = oracle.bitpack_pm1(a), oracle.bitpack_pm1(w)
    acc = oracle.bconv2d_acc(a, w, (s, s), padding)
    kw = dict(in_c=Cin, stride=(s, s), padding=padding)
    got = run_bconv(aw, ww, dict(kw, out_type=lce.OUT_INT32), kernel_choice=kernel_choice[0], packed=kernel_choice[1])
    np.testing.assert_array_equal(got, acc)
    K = k * k * Cin
    thr = np.rint(np.sqrt(K) * rng.standard_normal(Cout)).astype(np.int32)
    got = run_bconv(aw, ww, dict(kw, out_type=lce.OUT_BITPACKED), thr=thr, kernel_choice=kernel_choice[0], packed=kernel_choice[1])
    np.testing.assert_array_equal(got, oracle.transform_bits(acc, thr))
    mult = rng.uniform(0.5, 1.5, Cout).astype(np.float32)
    bias = (0.1 * rng.standard_normal(Cout)).astype(np.float32)
    for act in (lce.ACT_NONE, lce.ACT_RELU):
        got = run_bconv(aw, ww, dict(kw, out_type=lce.OUT_FLOAT32, activation=act), mult=mult, bias=bias,
                        kernel_choice=kernel_choice[0], packed=kernel_choice[1])
        assert float_close(got, acc, mult, bias, act) == 0  # goal: bit-identical floats


@pytest.mark.parametrize("kernel_choice", KERNELS, ids=KERNEL_IDS)
def test_saturated_thresholds_and_pad_bits(kernel_choice):
    rng = np.random.default_rng(77)
    a, w = rand_pm1(rng, (1, 6, 6, 64)), rand_pm1(rng, (40, 3, 3, 64))
    aw, ww = oracle.bitpack_pm1(a), oracle.bitpack_pm1(w)
    lo = np.full(40, np.iinfo(np.int32).min, np.int32)
    hi = np.full(40, np.iinfo(np.int32).max, np.int32)
    kw = dict(in_c=64, out_type=lce.OUT_BITPACKED)
    assert not run_bconv(aw, ww, kw, thr=lo, kernel_choice=kernel_choice[0], packed=kernel_choice[1]).any()
    ones = run_bconv(aw, ww, kw, thr=hi, kernel_choice=kernel_choice[0], packed=kernel_choice[1])
    assert np.all(ones[..., 0] == 0xFFFFFFFF) and np.all(ones[..., 1] == 0xFF)


# ---- tensor-core formulation (tcgen05 kind::mxf4 on +-1 / 0 e2m1 values): same integers, same bits ------

TENSOR_SHAPES = [
    # N, H, W, Cin, Cout  (3x3, stride 1, one-padding)
    (1, 7, 7, 64, 64), (2, 14, 14, 64, 64), (3, 9, 11, 70, 45), (1, 28, 28, 128, 128), (2, 7, 7, 512, 96),
    (1, 56, 56, 64, 64), (2, 14, 14, 256, 256), (1, 5, 5, 32, 300), (4, 7, 7, 512, 512), (2, 9, 9, 320, 40),
    (1, 1, 1, 3, 1), (5, 3, 40, 96, 130),
    # bit-packed output with Cout <= 128 and few input words: the pixels-as-N schedule, several tiles and images
    (2, 30, 30, 32, 128), (6, 20, 17, 64, 100), (1, 80, 80, 33, 33), (3, 40, 3, 96, 64),
    # float / int32 output with Cout <= 64, a multiple of 4: the same schedule with the shared-memory stage
    (2, 20, 20, 64, 48), (1, 30, 30, 32, 8), (4, 16, 16, 40, 60), (1, 12, 12, 64, 4), (3, 33, 31, 64, 32),
    # several tiles per CTA (more than 148 x 224 positions), three channel blocks, odd channel-word counts
    (40, 30, 30, 64, 64), (24, 28, 28, 96, 300), (9, 56, 56, 160, 64),
]


@pytest.mark.parametrize("shape", TENSOR_SHAPES)
def test_tensor_core_kernel_matches_oracle(shape):
    N, H, W, Cin, Cout = shape
    rng = np.random.default_rng(abs(hash(shape)) % 2**32)
    a, w = rand_pm1(rng, (N, H, W, Cin)), rand_pm1(rng, (Cout, 3, 3, Cin))
    aw, ww = oracle.bitpack_pm1(a), oracle.bitpack_pm1(w)
    acc = oracle.bconv2d_acc(a, w, (1, 1), lce.PAD_SAME_ONE)
    kw = dict(in_c=Cin, padding=lce.PAD_SAME_ONE)
    got = run_bconv(aw, ww, dict(kw, out_type=lce.OUT_INT32), kernel_choice=lce.KERNEL_TENSOR, packed=True)
    np.testing.assert_array_equal(got, acc)
    thr = np.rint(np.sqrt(9 * Cin) * rng.standard_normal(Cout)).astype(np.int32)
    got = run_bconv(aw, ww, dict(kw, out_type=lce.OUT_BITPACKED), thr=thr, kernel_choice=lce.KERNEL_TENSOR, packed=True)
    np.testing.assert_array_equal(got, oracle.transform_bits(acc, thr))
    mult = rng.uniform(0.5, 1.5, Cout).astype(np.float32)
    bias = (0.1 * rng.standard_normal(Cout)).astype(np.float32)
    for act in (lce.ACT_NONE, lce.ACT_RELU):
        got = run_bconv(aw, ww, dict(kw, out_type=lce.OUT_FLOAT32, activation=act), mult=mult, bias=bias,
                        kernel_choice=lce.KERNEL_TENSOR, packed=True)
        assert float_close(got, acc, mult, bias, act) == 0
    assert lce.lce_device_status() == 0  # no bounded wait gave up


def test_tensor_core_kernel_rejects_what_it_does_not_cover():
    z = torch.zeros(8 * 8 * 2, dtype=torch.int32, device=DEV)
    w = torch.zeros(64 * 9 * 2, dtype=torch.int32, device=DEV)
    # plain weights: the kernel needs the operand image made at load time
    desc = lce.make_desc(1, 8, 8, 64, 64, (3, 3), (1, 1), lce.PAD_SAME_ONE, lce.OUT_INT32, kernel_choice=lce.KERNEL_TENSOR)
    with pytest.raises(lce.LceError) as e:
        lce.lce_bconv2d(desc, z, w)
    assert e.value.status == 2
    # stride 3
    desc = lce.make_desc(1, 8, 8, 64, 64, (3, 3), (3, 3), lce.PAD_SAME_ONE, lce.OUT_INT32, lce.ACT_NONE, lce.KERNEL_TENSOR, 1)
    with pytest.raises(lce.LceError) as e:
        lce.lce_bconv2d(desc, z, lce.lce_bconv2d_pack_weights(desc, w))
    assert e.value.status == 2


# ---- config 1 and batch-reduced versions of configs 2, 3 ------------------------------------

def conv_case(config, first_index, spec, kernel_choice=(lce.KERNEL_AUTO, True)):
    t = wl.conv_tensors(config, first_index, spec)
    x = wl.activations(config, 0, (spec.batch, spec.in_h, spec.in_w, spec.in_c))
    a_words_oracle = oracle.bitpack(x)
    a_words_gpu = words_to_host(lce.lce_bitpack(to_dev(x)))
    np.testing.assert_array_equal(a_words_gpu, a_words_oracle)
    w_words = words_to_host(lce.pack_weights(to_dev(t.w_pm1)))
    np.testing.assert_array_equal(w_words, oracle.bitpack_pm1(t.w_pm1))
    acc = oracle.bconv2d_acc(oracle.sign(x), t.w_pm1, (spec.stride, spec.stride), spec.padding)
    kw = dict(in_c=spec.in_c, stride=(spec.stride, spec.stride), padding=spec.padding, out_type=spec.out_type)
    if spec.out_type == wl.OUT_FLOAT32:
        got = run_bconv(a_words_gpu, w_words, kw, mult=t.multiplier, bias=t.bias, kernel_choice=kernel_choice[0], packed=kernel_choice[1])
        assert float_close(got, acc, t.multiplier, t.bias) == 0
    else:
        got = run_bconv(a_words_gpu, w_words, kw, thr=t.thresholds, kernel_choice=kernel_choice[0], packed=kernel_choice[1])
        np.testing.assert_array_equal(got, oracle.transform_bits(acc, t.thresholds))


@pytest.mark.parametrize("kernel_choice", KERNELS, ids=KERNEL_IDS)
def test_config1_single_conv(kernel_choice):
    conv_case(1, 1, wl.config1_spec(), kernel_choice)


@pytest.mark.parametrize("spec", wl.config2_specs(batch=4) + wl.config3_specs(batch=4), ids=lambda s: s.name)
def test_config2_config3_shapes_small_batch(spec):
    conv_case(2, 1, spec)


# ---- LceQuantize fused into the convolution's loader -----------------------------------------

F32_SHAPES = [
    # N, H, W, Cin, Cout, k, s
    (1, 14, 14, 64, 64, 3, 1), (2, 9, 11, 70, 45, 3, 1), (1, 17, 13, 96, 33, 3, 2), (3, 8, 8, 33, 64, 5, 1),
    (1, 57, 9, 32, 64, 3, 1), (2, 16, 16, 256, 32, 5, 2), (1, 5, 5, 130, 8, 3, 1), (1, 30, 33, 40, 70, 3, 1),
]


@pytest.mark.parametrize("padding", [lce.PAD_VALID, lce.PAD_SAME_ONE, lce.PAD_SAME_ZERO])
@pytest.mark.parametrize("shape", F32_SHAPES)
def test_float_input_conv_matches_bitpack_then_conv(shape, padding):
    N, H, W, Cin, Cout, k, s = shape
    rng = np.random.default_rng(abs(hash((shape, padding, "f32"))) % 2**32)
    x = rng.standard_normal((N, H, W, Cin)).astype(np.float32)
    x[rng.random(x.shape) < 0.05] = 0.0      # sign(0) = +1
    x[rng.random(x.shape) < 0.02] = -0.0     # a negative zero is not negative
    w = rand_pm1(rng, (Cout, k, k, Cin))
    acc = oracle.bconv2d_acc(oracle.sign(x), w, (s, s), padding)
    ww = to_dev_words(oracle.bitpack_pm1(w))
    for packed in (0, 1):
        desc = lambda ot, act=lce.ACT_NONE: lce.make_desc(N, H, W, Cin, Cout, (k, k), (s, s), padding, ot, act, lce.KERNEL_AUTO, packed)
        wd = lce.lce_bconv2d_pack_weights(desc(lce.OUT_INT32), ww) if packed else ww
        got = lce.lce_bconv2d_f32(desc(lce.OUT_INT32), to_dev(x), wd).cpu().numpy()
        np.testing.assert_array_equal(got, acc)
        thr = np.rint(np.sqrt(k * k * Cin) * rng.standard_normal(Cout)).astype(np.int32)
        got = words_to_host(lce.lce_bconv2d_f32(desc(lce.OUT_BITPACKED), to_dev(x), wd, thresholds=to_dev(thr)))
        np.testing.assert_array_equal(got, oracle.transform_bits(acc, thr))
        mult = rng.uniform(0.5, 1.5, Cout).astype(np.float32)
        bias = (0.1 * rng.standard_normal(Cout)).astype(np.float32)
        got = lce.lce_bconv2d_f32(desc(lce.OUT_FLOAT32, lce.ACT_RELU), to_dev(x), wd, to_dev(mult), to_dev(bias)).cpu().numpy()
        assert float_close(got, acc, mult, bias, lce.ACT_RELU) == 0


def test_float_input_conv_config1_and_unsupported_shapes():
    spec = wl.config1_spec()
    t = wl.conv_tensors(1, 1, spec)
    x = wl.activations(1, 0, (spec.batch, spec.in_h, spec.in_w, spec.in_c))
    acc = oracle.bconv2d_acc(oracle.sign(x), t.w_pm1, (spec.stride, spec.stride), spec.padding)
    desc = lce.make_desc(spec.batch, spec.in_h, spec.in_w, spec.in_c, spec.out_c, (3, 3), (1, 1), spec.padding, spec.out_type)
    ww = to_dev_words(oracle.bitpack_pm1(t.w_pm1))
    if spec.out_type == wl.OUT_FLOAT32:
        got = lce.lce_bconv2d_f32(desc, to_dev(x), ww, to_dev(t.multiplier), to_dev(t.bias)).cpu().numpy()
        assert float_close(got, acc, t.multiplier, t.bias) == 0
    else:
        got = words_to_host(lce.lce_bconv2d_f32(desc, to_dev(x), ww, thresholds=to_dev(t.thresholds)))
        np.testing.assert_array_equal(got, oracle.transform_bits(acc, t.thresholds))
    # a 1x1 filter is outside the fused loader's coverage: status UNSUPPORTED, nothing launched
    d1 = lce.make_desc(1, 4, 4, 64, 8, (1, 1), (1, 1), lce.PAD_VALID, lce.OUT_INT32)
    with pytest.raises(lce.LceError) as e:
        lce.lce_bconv2d_f32(d1, torch.zeros(4 * 4 * 64, device=DEV), torch.zeros(8 * 2, dtype=torch.int32, device=DEV))
    assert e.value.status == 2


# ---- LceBMaxPool2d, add -------------------------------------------------------------------

@pytest.mark.parametrize("shape,pool,stride,padding", [
    ((2, 8, 8, 64), (2, 2), (2, 2), lce.PAD_VALID), ((1, 7, 9, 45), (3, 3), (2, 2), lce.PAD_SAME_ONE),
    ((3, 5, 6, 130), (2, 3), (1, 2), lce.PAD_VALID), ((2, 56, 56, 64), (2, 2), (2, 2), lce.PAD_VALID),
    ((1, 9, 9, 33), (3, 3), (1, 1), lce.PAD_SAME_ONE)])
def test_bmaxpool_matches_oracle(shape, pool, stride, padding):
    rng = np.random.default_rng(sum(shape))
    C = shape[-1]
    words = oracle.bitpack(rng.standard_normal(shape).astype(np.float32))
    got = words_to_host(lce.lce_bmaxpool(to_dev_words(words), C, pool, stride, padding))
    np.testing.assert_array_equal(got, oracle.bmaxpool(words, C, pool, stride, padding))


@pytest.mark.parametrize("n", [1, 3, 4, 1023, 4096, 100001])
def test_add_matches_oracle(n):
    rng = np.random.default_rng(n)
    a = (rng.standard_normal(n) * 100).astype(np.float32)
    b = rng.standard_normal(n).astype(np.float32)
    got = lce.lce_add_f32(to_dev(a), to_dev(b)).cpu().numpy()
    np.testing.assert_array_equal(got, oracle.add_f32(a, b))


def test_host_buffer_entry_point_matches_device_entry_point():
    spec = wl.with_batch(wl.config2_specs()[1], 2)  # 56x56x64 bit-packed, batch 2
    t = wl.conv_tensors(2, 1, spec)
    x = wl.activations(2, 0, (spec.batch, spec.in_h, spec.in_w, spec.in_c))
    aw, ww = oracle.bitpack(x), oracle.bitpack_pm1(t.w_pm1)
    desc = lce.make_desc(spec.batch, spec.in_h, spec.in_w, spec.in_c, spec.out_c, out_type=lce.OUT_BITPACKED)
    ws = torch.empty(lce.lce_bconv2d_host_workspace_bytes(desc), dtype=torch.uint8, device=DEV)
    h_in = torch.from_numpy(aw.view(np.int32)).pin_memory()
    h_w = torch.from_numpy(ww.view(np.int32)).pin_memory()
    h_thr = torch.from_numpy(t.thresholds).pin_memory()
    h_out = torch.empty((spec.batch, spec.out_h, spec.out_w, 2), dtype=torch.int32).pin_memory()
    lce.lce_bconv2d_host(desc, h_in, h_w, None, None, h_thr, h_out, ws)
    acc = oracle.bconv2d_acc(oracle.sign(x), t.w_pm1, (1, 1), spec.padding)
    np.testing.assert_array_equal(h_out.numpy().view(np.uint32), oracle.transform_bits(acc, t.thresholds))
    with pytest.raises(lce.LceError) as e:
        lce.lce_bconv2d_host(desc, h_in, h_w, None, None, h_thr, h_out, ws[:1024])
    assert e.value.status == 6


def test_async_host_entry_point_on_two_streams_matches_oracle():
    # two layers in flight on two streams, each with its own workspace; results read after synchronising
    jobs = []
    streams = [torch.cuda.Stream(device=DEV), torch.cuda.Stream(device=DEV)]
    for j, base in enumerate((wl.config2_specs()[0], wl.config2_specs()[3])):  # float 56x56x64, bits 28x28x128
        spec = wl.with_batch(base, 2)
        t = wl.conv_tensors(2, 1 + 4 * j, spec)
        x = wl.activations(2, j, (spec.batch, spec.in_h, spec.in_w, spec.in_c))
        desc = lce.make_desc(spec.batch, spec.in_h, spec.in_w, spec.in_c, spec.out_c, out_type=spec.out_type)
        ws = torch.empty(lce.lce_bconv2d_host_workspace_bytes(desc), dtype=torch.uint8, device=DEV)
        h_in = torch.from_numpy(oracle.bitpack(x).view(np.int32)).pin_memory()
        h_w = torch.from_numpy(oracle.bitpack_pm1(t.w_pm1).view(np.int32)).pin_memory()
        is_f = spec.out_type == wl.OUT_FLOAT32
        last = spec.out_c if is_f else (spec.out_c + 31) // 32
        h_out = torch.empty((spec.batch, spec.out_h, spec.out_w, last), dtype=torch.float32 if is_f else torch.int32).pin_memory()
        h_m = torch.from_numpy(t.multiplier).pin_memory() if is_f else None
        h_b = torch.from_numpy(t.bias).pin_memory() if is_f else None
        h_t = None if is_f else torch.from_numpy(t.thresholds).pin_memory()
        jobs.append((spec, t, x, desc, ws, h_in, h_w, h_m, h_b, h_t, h_out))
    torch.cuda.synchronize()
    for j, (spec, t, x, desc, ws, h_in, h_w, h_m, h_b, h_t, h_out) in enumerate(jobs):
        with torch.cuda.stream(streams[j]):
            lce.lce_bconv2d_host_async(desc, h_in, h_w, h_m, h_b, h_t, h_out, ws)
    for s in streams:
        s.synchronize()
    for spec, t, x, desc, ws, h_in, h_w, h_m, h_b, h_t, h_out in jobs:
        acc = oracle.bconv2d_acc(oracle.sign(x), t.w_pm1, (1, 1), spec.padding)
        if spec.out_type == wl.OUT_FLOAT32:
            assert float_close(h_out.numpy(), acc, t.multiplier, t.bias) == 0
        else:
            np.testing.assert_array_equal(h_out.numpy().view(np.uint32), oracle.transform_bits(acc, t.thresholds))


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_seeded_random_shapes_through_the_dispatcher(seed):
    """40 random layer shapes per seed (filter 1/3/5, stride 1/2, all paddings, ragged channel counts,
    plain or load-time packed weights): whatever kernel and work split the dispatcher picks, int32,
    bit-packed and float outputs equal the oracle's."""
    rng = np.random.default_rng(seed)
    done = 0
    while done < 40:
        k, s = int(rng.choice([1, 3, 3, 5])), int(rng.choice([1, 1, 2]))
        N, H, W = int(rng.integers(1, 7)), int(rng.integers(1, 70)), int(rng.integers(1, 70))
        Cin = int(rng.choice([rng.integers(1, 40), rng.integers(1, 300), 32, 64, 96, 128]))
        Cout = int(rng.choice([rng.integers(1, 40), rng.integers(1, 300), 32, 64, 96, 160]))
        padding = int(rng.integers(0, 3))
        if (padding == lce.PAD_VALID and (H < k or W < k)) or N * H * W * Cout * k * k * Cin > 2e9:
            continue
        done += 1
        packed = bool(rng.integers(0, 2))
        a, w = rand_pm1(rng, (N, H, W, Cin)), rand_pm1(rng, (Cout, k, k, Cin))
        aw, ww = oracle.bitpack_pm1(a), oracle.bitpack_pm1(w)
        acc = oracle.bconv2d_acc(a, w, (s, s), padding)
        kw = dict(in_c=Cin, stride=(s, s), padding=padding)
        where = f"N={N} H={H} W={W} Cin={Cin} Cout={Cout} k={k} s={s} padding={padding} packed={packed}"
        got = run_bconv(aw, ww, dict(kw, out_type=lce.OUT_INT32), packed=packed)
        assert np.array_equal(got, acc), where
        thr = np.rint(np.sqrt(k * k * Cin) * rng.standard_normal(Cout)).astype(np.int32)
        got = run_bconv(aw, ww, dict(kw, out_type=lce.OUT_BITPACKED), thr=thr, packed=packed)
        assert np.array_equal(got, oracle.transform_bits(acc, thr)), where
        mult = rng.uniform(0.5, 1.5, Cout).astype(np.float32)
        bias = (0.1 * rng.standard_normal(Cout)).astype(np.float32)
        act = int(rng.integers(0, 2))
        got = run_bconv(aw, ww, dict(kw, out_type=lce.OUT_FLOAT32, activation=act), mult=mult, bias=bias, packed=packed)
        assert float_close(got, acc, mult, bias, act) == 0, where


# ---- thresholds at and beyond the ends of the accumulator range --------------------------------------

@pytest.mark.parametrize("shape", [
    # N, H, W, Cin, Cout, k, stride, padding
    (2, 12, 12, 64, 64, 3, 1, lce.PAD_SAME_ONE), (1, 9, 10, 70, 40, 3, 2, lce.PAD_VALID), (2, 8, 8, 32, 96, 5, 1, lce.PAD_SAME_ONE),
    (1, 6, 6, 128, 64, 1, 1, lce.PAD_VALID), (1, 7, 7, 64, 33, 3, 1, lce.PAD_SAME_ZERO), (1, 4, 4, 3700, 8, 3, 1, lce.PAD_SAME_ONE),
])
@pytest.mark.parametrize("packed", [False, True])
def test_thresholds_at_the_ends_of_the_accumulator_range(shape, packed):
    """Section 3.2: the bit-packed output is acc < threshold[c].  Accumulators of +K and -K are forced
    (a channel equal to the all-ones input, its complement) and thresholds sit on, next to and far
    beyond both ends, including INT32_MIN and INT32_MAX."""
    N, H, W, Cin, Cout, k, s, padding = shape
    rng = np.random.default_rng(abs(hash(shape)) % 2**32)
    a = rand_pm1(rng, (N, H, W, Cin))
    a[0] = 1                                   # image 0: all +1
    w = rand_pm1(rng, (Cout, k, k, Cin))
    w[0::4] = 1                                # acc = +K wherever the window lies inside image 0 (or on one-padding)
    w[1::4] = -1                               # acc = -K there
    K = k * k * Cin
    edge = [-K - 2, -K - 1, -K, -K + 1, -K + 2, -1, 0, 1, K - 2, K - 1, K, K + 1, K + 2, -2**31, 2**31 - 1, -2**31 + 1, 2**31 - 2,
            -65536, 65536, -32768, 32767]
    thr = np.array([edge[(c // 4 + 5 * (c % 4)) % len(edge)] for c in range(Cout)], dtype=np.int64)
    thr[2::4] = rng.integers(-K - 3, K + 4, size=len(thr[2::4]))
    thr = thr.astype(np.int32)
    acc = oracle.bconv2d_acc(a, w, (s, s), padding)
    assert acc.max() == K and (acc.min() == -K)
    got = run_bconv(oracle.bitpack_pm1(a), oracle.bitpack_pm1(w), dict(in_c=Cin, stride=(s, s), padding=padding, out_type=lce.OUT_BITPACKED),
                    thr=thr, packed=packed)
    np.testing.assert_array_equal(got, oracle.transform_bits(acc, thr))


def test_plan_object_runs_like_the_direct_call_and_inside_a_cuda_graph():
    """lce_bconv2d_plan_create / lce_plan_run: the same launch as lce_bconv2d, capturable in a graph."""
    rng = np.random.default_rng(77)
    N, H, W, Cin, Cout = 3, 13, 11, 96, 72
    a, w = rand_pm1(rng, (N, H, W, Cin)), rand_pm1(rng, (Cout, 3, 3, Cin))
    acc = oracle.bconv2d_acc(a, w, (1, 1), lce.PAD_SAME_ONE)
    thr = np.rint(np.sqrt(9 * Cin) * rng.standard_normal(Cout)).astype(np.int32)
    desc = lce.make_desc(N, H, W, Cin, Cout, (3, 3), (1, 1), lce.PAD_SAME_ONE, lce.OUT_BITPACKED, lce.ACT_NONE, lce.KERNEL_AUTO, 1)
    a_dev, w_dev = to_dev_words(oracle.bitpack_pm1(a)), to_dev_words(oracle.bitpack_pm1(w))
    w_img = lce.lce_bconv2d_pack_weights(desc, w_dev)
    plan = lce.lce_bconv2d_plan_create(desc, a_dev, w_img, thresholds=to_dev(thr))
    want = oracle.transform_bits(acc, thr)
    out = lce.lce_plan_run(plan)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out.cpu().numpy().view(np.uint32), want)
    out.zero_()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            lce.lce_plan_run(plan)
        graph.replay()
        stream.synchronize()
    np.testing.assert_array_equal(out.cpu().numpy().view(np.uint32), want)
    lce.lce_plan_destroy(plan)
