"""Configs 4 and 5 (residual block stack, ImageNet-shaped body) at reduced batch: every buffer of
the GPU chain against the oracle chain (layer by layer and therefore end to end), bit-exact --
float tensors included, since one differing float could flip a sign bit downstream."""
import numpy as np
import pytest
import torch

import lce_workloads as wl
from chain_oracle import run_chain_oracle
from chains import Chain

pytestmark = pytest.mark.gpu


def compare_all(chain, ref):
    torch.cuda.synchronize()
    for name, t in chain.buffers.items():
        got = t.cpu().numpy()
        want = ref[name]
        if got.dtype == np.int32:
            got = got.view(np.uint32)
        assert got.shape == want.shape, name
        assert np.array_equal(got, want), f"buffer {name} differs"


def test_config4_block_stack_batch2():
    steps = wl.config4_steps(batch=2)
    x = wl.activations(4, 0, (2, 56, 56, 64))
    chain = Chain(steps, 4)
    chain.set_input("X0", x)
    chain.run()
    ref = run_chain_oracle(steps, 4, {"X0": x})
    compare_all(chain, ref)
    assert chain.buffers["Y3"].shape == (2, 7, 7, 512)
    # 7 bitpack + 11 bconv + 4 add + 3 bmaxpool
    assert chain.launches == 25


def test_config4_fused_chain_equals_unfused_chain():
    """Shortcut add and re-quantize folded into the convs: every tensor the fused chain writes equals
    the oracle's unfused chain (same names, same parameters)."""
    x = wl.activations(4, 0, (2, 56, 56, 64))
    fused = wl.config4_fused_steps(batch=2)
    chain = Chain(fused, 4)
    chain.set_input("X0", x)
    chain.run()
    ref_unfused = run_chain_oracle(wl.config4_steps(batch=2), 4, {"X0": x})
    ref_fused = run_chain_oracle(fused, 4, {"X0": x})
    compare_all(chain, ref_fused)
    compare_all(chain, {k: ref_unfused[k] for k in chain.buffers})
    assert chain.launches == 15


def test_fused_conv_on_ragged_shape():
    import oracle
    import paper_2011_09398_b200 as lce
    rng = np.random.default_rng(5)
    N, H, W, Cin, Cout = 2, 9, 7, 70, 45
    a = (2 * rng.integers(0, 2, size=(N, H, W, Cin)) - 1).astype(np.int8)
    w = (2 * rng.integers(0, 2, size=(Cout, 3, 3, Cin)) - 1).astype(np.int8)
    mult = rng.uniform(0.5, 1.5, Cout).astype(np.float32)
    bias = rng.standard_normal(Cout).astype(np.float32)
    res = rng.standard_normal((N, H, W, Cout)).astype(np.float32) * 30
    y = oracle.add_f32(oracle.transform_float(oracle.bconv2d_acc(a, w), mult, bias), res)
    dev = "cuda:0"
    desc = lce.make_desc(N, H, W, Cin, Cout, out_type=lce.OUT_FLOAT32)
    t = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    of = torch.empty((N, H, W, Cout), dtype=torch.float32, device=dev)
    op = torch.empty((N, H, W, 2), dtype=torch.int32, device=dev)
    lce.lce_bconv2d_fused(desc, t(oracle.bitpack_pm1(a).view(np.int32)), t(oracle.bitpack_pm1(w).view(np.int32)),
                          t(mult), t(bias), t(res), of, op)
    assert np.array_equal(of.cpu().numpy(), y)
    assert np.array_equal(op.cpu().numpy().view(np.uint32), oracle.bitpack(y))


def test_config5_body_batch2():
    steps = wl.config5_steps(batch=2)
    x = wl.activations(5, 0, (2, 224, 224, 3))
    chain = Chain(steps, 5)
    chain.set_input("X", x)
    chain.run()
    ref = run_chain_oracle(steps, 5, {"X": x})
    compare_all(chain, ref)
    assert chain.buffers["T17"].shape == (2, 7, 7, 512)
    assert sum(1 for s in steps if s.kind == "bconv") == 17


def test_small_odd_chain_with_ragged_channels():
    # a miniature body with channel counts that are not multiples of 32 and odd image sizes
    steps = wl.config5_steps(batch=3, size=30, in_c=3, stem_c=24, widths=(40, 72), per_stage=2)
    x = wl.activations(5, 0, (3, 30, 30, 3))
    chain = Chain(steps, 5)
    chain.set_input("X", x)
    chain.run()
    compare_all(chain, run_chain_oracle(steps, 5, {"X": x}))
