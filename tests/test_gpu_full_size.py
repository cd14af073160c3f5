"""GPU parity at the full benchmark sizes, every output element: configs 2 and 3 at batch 64 (the launch
configuration bench.py times: load-time packed weights, the kernel the dispatcher picks, and the integer
XOR/POPC kernel forced), config 4 at batch 128 and config 5 at batch 256 (every buffer of the chain).
The oracle computes each whole layer from the definition (a fraction of a second per layer on the host
cores); int32 and bit-packed outputs must be identical, float outputs must not differ in a single value
(the stated tolerance is checked first).  Around that: range-edge samples as a fast first assertion and
the weight-complement property of the accumulators (Section 2: the dot product of +-1 vectors is odd
in either factor).
"""
import numpy as np
import pytest
import torch

import lce_workloads as wl
import oracle
import paper_2011_09398_b200 as lce
from chain_oracle import run_chain_oracle
from chains import Chain
from gpu_util import to_dev, to_dev_words

pytestmark = pytest.mark.gpu


def edge_samples(rng, spec, count=400):
    """Random outputs plus every corner of the tensor and the pixels on either side of the places where a
    CTA's share of the work can begin or end."""
    N, OH, OW, Co = spec.batch, spec.out_h, spec.out_w, spec.out_c
    idx = np.stack([rng.integers(0, N, count), rng.integers(0, OH, count), rng.integers(0, OW, count),
                    rng.integers(0, Co, count)], axis=1)
    corners = [(n, oh, ow, o) for n in (0, N - 1) for oh in (0, OH - 1) for ow in (0, OW - 1) for o in (0, Co // 2, Co - 1)]
    M = N * OH * OW
    edges = []
    for k in range(1, 148, 7):
        for m in {(M * k // 148) // 32 * 32 + d for d in (-1, 0, 1, 31, 32, 63, 64)}:
            if 0 <= m < M:
                edges.append((m // (OH * OW), (m // OW) % OH, m % OW, int(rng.integers(0, Co))))
    return np.concatenate([idx, np.array(corners), np.array(edges)]).astype(np.int32)


def gpu_layer(spec, t, a_words, w_words, kernel_choice, out_type):
    desc = lce.make_desc(spec.batch, spec.in_h, spec.in_w, spec.in_c, spec.out_c, (spec.kernel, spec.kernel),
                         (spec.stride, spec.stride), spec.padding, out_type, lce.ACT_NONE, kernel_choice, 1)
    wd = lce.lce_bconv2d_pack_weights(desc, w_words)
    mult = to_dev(t.multiplier) if out_type == lce.OUT_FLOAT32 else None
    bias = to_dev(t.bias) if out_type == lce.OUT_FLOAT32 else None
    thr = to_dev(t.thresholds) if out_type == lce.OUT_BITPACKED else None
    return lce.lce_bconv2d(desc, a_words, wd, mult, bias, thr), lce.lce_bconv2d_plan(desc)["kernel"]


def assert_layer_equal(spec, t, acc, out, out_type, rng):
    host = out.cpu().numpy()
    idx = edge_samples(rng, spec)
    n, oh, ow, o = idx.T
    if out_type == lce.OUT_INT32:
        np.testing.assert_array_equal(host[n, oh, ow, o], acc[n, oh, ow, o])       # fast first look
        np.testing.assert_array_equal(host, acc)
    elif out_type == lce.OUT_BITPACKED:
        words = host.view(np.uint32)
        np.testing.assert_array_equal((words[n, oh, ow, o // 32] >> (o % 32).astype(np.uint32)) & 1,
                                      (acc[n, oh, ow, o] < t.thresholds[o]).astype(np.uint32))
        np.testing.assert_array_equal(words, oracle.transform_bits(acc, t.thresholds))
    else:
        want = oracle.transform_float(acc, t.multiplier, t.bias)
        a64 = acc.astype(np.float64)
        tol = 1e-6 * (np.abs(a64 * t.multiplier) + np.abs(t.bias))  # the stated tolerance; one fp32 rounding is 6e-8
        assert np.all(np.abs(host.astype(np.float64) - (a64 * t.multiplier.astype(np.float64) + t.bias.astype(np.float64))) <= tol)
        assert int((host != want).sum()) == 0                      # the goal: not one differing float


FULL = [(2, 1 + 4 * i, s) for i, s in enumerate(wl.config2_specs())] + [(3, 1 + 4 * i, s) for i, s in enumerate(wl.config3_specs())]


@pytest.mark.parametrize("config,first,spec", FULL, ids=[s.name for _, _, s in FULL])
def test_full_size_layer_every_element_against_oracle(config, first, spec):
    """All outputs of the layer at batch 64, through the kernel AUTO picks for load-time packed weights
    (the tensor-core kernel at these sizes) and through the integer XOR/POPC kernel."""
    rng = np.random.default_rng(config * 1000 + first)
    t = wl.conv_tensors(config, first, spec)
    x = wl.activations(config, 0, (spec.batch, spec.in_h, spec.in_w, spec.in_c))
    acc = oracle.bconv2d_acc(oracle.sign(x), t.w_pm1, (spec.stride, spec.stride), spec.padding)
    a_words = lce.lce_bitpack(to_dev(x))
    w_words = to_dev_words(oracle.bitpack_pm1(t.w_pm1))
    picked = set()
    for kernel_choice in (lce.KERNEL_AUTO, lce.KERNEL_TILED):
        out, kernel = gpu_layer(spec, t, a_words, w_words, kernel_choice, spec.out_type)
        picked.add(kernel)
        assert_layer_equal(spec, t, acc, out, spec.out_type, rng)
    assert picked == {lce.KERNEL_TENSOR, lce.KERNEL_TILED}
    assert lce.lce_device_status() == 0


@pytest.mark.parametrize("kernel_choice", [lce.KERNEL_TENSOR, lce.KERNEL_TILED], ids=["tensor", "tiled"])
@pytest.mark.parametrize("spec", wl.config2_specs()[::2] + wl.config3_specs()[:2], ids=lambda s: s.name)
def test_full_size_accumulators_and_weight_complement(spec, kernel_choice):
    t = wl.conv_tensors(2, 1, spec)
    x = wl.activations(2, 0, (spec.batch, spec.in_h, spec.in_w, spec.in_c))
    acc_ref = oracle.bconv2d_acc(oracle.sign(x), t.w_pm1, (spec.stride, spec.stride), spec.padding)
    a_words = lce.lce_bitpack(to_dev(x))
    w_words = to_dev_words(oracle.bitpack_pm1(t.w_pm1))
    acc, _ = gpu_layer(spec, t, a_words, w_words, kernel_choice, lce.OUT_INT32)
    np.testing.assert_array_equal(acc.cpu().numpy(), acc_ref)
    assert spec.in_c % 32 == 0  # no pad bits to keep at zero
    acc_flipped, _ = gpu_layer(spec, t, a_words, torch.bitwise_not(w_words), kernel_choice, lce.OUT_INT32)
    assert torch.equal(acc_flipped, -acc)
    K = spec.K
    assert int(acc.abs().max().item()) <= K and bool(((acc + K) % 2 == 0).all().item())


def test_full_size_largest_sweep_layer_5x5_sampled():
    """The paper's largest sweep layer (64x64x256, 5x5) at batch 64 is 429 G MAC: sampled here (a few
    thousand outputs, corners and range edges), every element at batch 4 below."""
    spec = [s for s in wl.sweep_specs(64) if s.name == "sweep_64x64x256_k5"][0]
    rng = np.random.default_rng(55)
    t = wl.conv_tensors(6, 1, spec)
    x = wl.activations(6, 0, (spec.batch, spec.in_h, spec.in_w, spec.in_c))
    a_sign = oracle.sign(x)
    a_words = lce.lce_bitpack(to_dev(x))
    w_words = to_dev_words(oracle.bitpack_pm1(t.w_pm1))
    idx = edge_samples(rng, spec, 3000)
    acc = oracle.bconv2d_acc_at(a_sign, t.w_pm1, idx, (1, 1), spec.padding)
    n, oh, ow, o = idx.T
    for kernel_choice in (lce.KERNEL_AUTO, lce.KERNEL_TILED):
        out, _ = gpu_layer(spec, t, a_words, w_words, kernel_choice, lce.OUT_INT32)
        np.testing.assert_array_equal(out.cpu().numpy()[n, oh, ow, o], acc)
    small = wl.with_batch(spec, 4)
    acc4 = oracle.bconv2d_acc(a_sign[:4], t.w_pm1, (1, 1), spec.padding)
    for kernel_choice in (lce.KERNEL_TENSOR, lce.KERNEL_TILED):
        out, _ = gpu_layer(small, t, a_words[:4].contiguous(), w_words, kernel_choice, spec.out_type)
        assert_layer_equal(small, t, acc4, out, spec.out_type, rng)


def compare_chain(chain, ref):
    torch.cuda.synchronize()
    for name, tensor in chain.buffers.items():
        got = tensor.cpu().numpy()
        want = ref[name]
        if got.dtype == np.int32:
            got = got.view(np.uint32)
        assert got.shape == want.shape, name
        assert np.array_equal(got, want), f"buffer {name} differs"


@pytest.mark.parametrize("fused", [False, True], ids=["25-launches", "fused-15-launches"])
def test_config4_block_stack_at_batch_128_every_buffer(fused):
    steps = wl.config4_fused_steps() if fused else wl.config4_steps()
    x = wl.activations(4, 0, (128, 56, 56, 64))
    chain = Chain(steps, 4)
    chain.set_input("X0", x)
    chain.run()
    compare_chain(chain, run_chain_oracle(steps, 4, {"X0": x}))
    assert chain.buffers["Y3"].shape == (128, 7, 7, 512)
    assert lce.lce_device_status() == 0


def test_config5_body_at_batch_256_every_buffer():
    steps = wl.config5_steps()
    x = wl.activations(5, 0, (256, 224, 224, 3))
    chain = Chain(steps, 5)
    chain.set_input("X", x)
    chain.run()
    compare_chain(chain, run_chain_oracle(steps, 5, {"X": x}))
    assert chain.buffers["T17"].shape == (256, 7, 7, 512)
    assert lce.lce_device_status() == 0
