"""GPU parity at the full benchmark sizes (batch 64, load-time packed weights, the kernel the
dispatcher picks: the launch configuration bench.py times).  The oracle cannot compute a whole
7.4-G-MAC layer in test time, so every layer is checked two ways:
  * sampled outputs: a few thousand (n, oh, ow, o) coordinates - random ones, every corner of the
    tensor, and the pixels on either side of the CTA range boundaries - each computed by the oracle
    from the definition, compared exactly (int32, bits) or within the float tolerance;
  * a property that holds at any size and covers every output: complementing every weight bit
    negates every accumulator (Section 2: the dot product of +-1 vectors is odd in either factor).
"""
import numpy as np
import pytest
import torch

import lce_workloads as wl
import oracle
import paper_2011_09398_b200 as lce
from gpu_util import DEV, to_dev, to_dev_words, words_to_host

pytestmark = pytest.mark.gpu

SAMPLES = 3000


def sample_indices(rng, spec):
    N, OH, OW, Co = spec.batch, spec.out_h, spec.out_w, spec.out_c
    idx = np.stack([rng.integers(0, N, SAMPLES), rng.integers(0, OH, SAMPLES), rng.integers(0, OW, SAMPLES),
                    rng.integers(0, Co, SAMPLES)], axis=1)
    corners = [(n, oh, ow, o) for n in (0, N - 1) for oh in (0, OH - 1) for ow in (0, OW - 1) for o in (0, Co // 2, Co - 1)]
    # flat pixels next to where a CTA's range can begin or end: multiples of 32 around M * k / 148
    M = N * OH * OW
    edges = []
    for k in range(1, 148, 7):
        for m in {(M * k // 148) // 32 * 32 + d for d in (-1, 0, 1, 31, 32, 63, 64)}:
            if 0 <= m < M:
                edges.append((m // (OH * OW), (m // OW) % OH, m % OW, int(rng.integers(0, Co))))
    return np.concatenate([idx, np.array(corners), np.array(edges)]).astype(np.int32)


def run_layer(config, first_index, spec, kernel_choice, packed, out_type=None):
    t = wl.conv_tensors(config, first_index, spec)
    x = wl.activations(config, 0, (spec.batch, spec.in_h, spec.in_w, spec.in_c))
    a_sign = oracle.sign(x)
    a_words = lce.lce_bitpack(to_dev(x))
    w_words = to_dev_words(oracle.bitpack_pm1(t.w_pm1))
    ot = spec.out_type if out_type is None else out_type
    desc = lce.make_desc(spec.batch, spec.in_h, spec.in_w, spec.in_c, spec.out_c, (spec.kernel, spec.kernel),
                         (spec.stride, spec.stride), spec.padding, ot, lce.ACT_NONE, kernel_choice, 1 if packed else 0)
    wd = lce.lce_bconv2d_pack_weights(desc, w_words) if packed else w_words
    mult = to_dev(t.multiplier) if ot == lce.OUT_FLOAT32 else None
    bias = to_dev(t.bias) if ot == lce.OUT_FLOAT32 else None
    thr = to_dev(t.thresholds) if ot == lce.OUT_BITPACKED else None
    out = lce.lce_bconv2d(desc, a_words, wd, mult, bias, thr)
    return t, a_sign, a_words, w_words, desc, out


def check_samples(spec, t, a_sign, out, ot, rng):
    idx = sample_indices(rng, spec)
    acc = oracle.bconv2d_acc_at(a_sign, t.w_pm1, idx, (spec.stride, spec.stride), spec.padding)
    n, oh, ow, o = idx.T
    host = out.cpu().numpy()
    if ot == lce.OUT_INT32:
        np.testing.assert_array_equal(host[n, oh, ow, o], acc)
    elif ot == lce.OUT_BITPACKED:
        words = host.view(np.uint32)[n, oh, ow, o // 32]
        np.testing.assert_array_equal((words >> (o % 32).astype(np.uint32)) & 1, (acc < t.thresholds[o]).astype(np.uint32))
    else:
        got = host[n, oh, ow, o]
        m, b = t.multiplier[o], t.bias[o]
        want = (acc.astype(np.float64) * m.astype(np.float64) + b.astype(np.float64))
        tol = 1e-6 * (np.abs(acc.astype(np.float64) * m) + np.abs(b))  # the stated tolerance; one fp32 rounding is 6e-8
        assert np.all(np.abs(got.astype(np.float64) - want) <= tol)


FULL = [(2, 1 + 4 * i, s) for i, s in enumerate(wl.config2_specs())] + [(3, 1 + 4 * i, s) for i, s in enumerate(wl.config3_specs())]


@pytest.mark.parametrize("config,first,spec", FULL, ids=[s.name for _, _, s in FULL])
def test_full_size_layer_sampled_against_oracle(config, first, spec):
    rng = np.random.default_rng(config * 1000 + first)
    t, a_sign, _, _, _, out = run_layer(config, first, spec, lce.KERNEL_AUTO, packed=True)
    check_samples(spec, t, a_sign, out, spec.out_type, rng)


@pytest.mark.parametrize("spec", wl.config2_specs()[1::2] + wl.config2_specs()[:1], ids=lambda s: s.name)
def test_full_size_tensor_core_layer_sampled_against_oracle(spec):
    rng = np.random.default_rng(abs(hash(spec.name)) % 2**32)
    t, a_sign, _, _, _, out = run_layer(2, 1, spec, lce.KERNEL_TENSOR, packed=False)
    check_samples(spec, t, a_sign, out, spec.out_type, rng)
    assert lce.lce_device_status() == 0


@pytest.mark.parametrize("kernel_choice,packed", [(lce.KERNEL_AUTO, True), (lce.KERNEL_TENSOR, False)], ids=["auto-packed", "tensor"])
@pytest.mark.parametrize("spec", wl.config2_specs()[::2], ids=lambda s: s.name)
def test_full_size_weight_complement_negates_every_accumulator(spec, kernel_choice, packed):
    t, a_sign, a_words, w_words, desc, acc = run_layer(2, 1, spec, kernel_choice, packed, out_type=lce.OUT_INT32)
    assert spec.in_c % 32 == 0  # no pad bits to keep at zero
    w_flipped = torch.bitwise_not(w_words)
    wd = lce.lce_bconv2d_pack_weights(desc, w_flipped) if packed else w_flipped
    acc_flipped = lce.lce_bconv2d(desc, a_words, wd)
    assert torch.equal(acc_flipped, -acc)
    # and the accumulators have the parity of K and stay within [-K, K]
    K = spec.K
    assert int(acc.abs().max().item()) <= K
    assert bool(((acc + K) % 2 == 0).all().item())
    check_samples(spec, t, a_sign, acc, lce.OUT_INT32, np.random.default_rng(7))


def test_full_size_largest_sweep_layer_5x5():
    spec = [s for s in wl.sweep_specs(64) if s.name == "sweep_64x64x256_k5"][0]
    rng = np.random.default_rng(55)
    t, a_sign, _, _, _, out = run_layer(6, 1, spec, lce.KERNEL_AUTO, packed=True)
    check_samples(spec, t, a_sign, out, spec.out_type, rng)
