"""Configs 4 and 5 (residual block stack, ImageNet-shaped body) at reduced batch: every buffer of
the GPU chain against the oracle chain (layer by layer and therefore end to end), bit-exact --
float tensors included, since one differing float could flip a sign bit downstream."""
import numpy as np
import pytest
import torch

import lce_workloads as wl
from chain_oracle import run_chain_oracle
from paper_2011_09398_b200.chains import Chain

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
