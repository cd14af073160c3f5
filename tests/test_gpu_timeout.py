"""A bounded device-side wait that runs out: reported to the host, surfaced by the next call, cleared by
the reset, and the library keeps working afterwards.  The wait that expires belongs to a tiny dedicated
kernel (lce_device_wait_probe: one thread waits, with the convolution kernels' own helper and a short
limit, on a barrier nobody arrives at); the convolution kernels' waits are never made to expire."""
import numpy as np
import pytest
import torch

import oracle
import paper_2011_09398_b200 as lce
from gpu_util import DEV, to_dev, to_dev_words

pytestmark = pytest.mark.gpu


def small_case():
    rng = np.random.default_rng(3)
    a = (2 * rng.integers(0, 2, size=(2, 9, 9, 64)) - 1).astype(np.int8)
    w = (2 * rng.integers(0, 2, size=(40, 3, 3, 64)) - 1).astype(np.int8)
    return a, w, oracle.bconv2d_acc(a, w)


def test_expired_wait_is_reported_by_the_next_call_and_cleared_by_the_reset():
    a, w, acc = small_case()
    aw, ww = to_dev_words(oracle.bitpack_pm1(a)), to_dev_words(oracle.bitpack_pm1(w))
    desc = lce.make_desc(2, 9, 9, 64, 40, out_type=lce.OUT_INT32, kernel_choice=lce.KERNEL_TENSOR, weights_packed=1)
    wp = lce.lce_bconv2d_pack_weights(desc, ww)
    assert lce.lce_device_status() == 0
    assert np.array_equal(lce.lce_bconv2d(desc, aw, wp).cpu().numpy(), acc)
    try:
        lce.lce_device_wait_probe(20_000)           # 20 microseconds: runs out, the kernel returns normally
        torch.cuda.synchronize()                    # no error, the context is intact
        assert lce.lce_device_status() == 1
        for forced in (lce.KERNEL_TENSOR, lce.KERNEL_AUTO):
            d = lce.make_desc(2, 9, 9, 64, 40, out_type=lce.OUT_INT32, kernel_choice=forced, weights_packed=1)
            with pytest.raises(lce.LceError) as e:  # nothing is launched while the status is set
                lce.lce_bconv2d(d, aw, wp)
            assert e.value.status == 5
        plan = lce.lce_bconv2d_plan_create(desc, aw, wp, None, None, None, torch.empty((2, 9, 9, 40), dtype=torch.int32, device=DEV))
        with pytest.raises(lce.LceError) as e:
            lce.lce_plan_run(plan)
        assert e.value.status == 5
    finally:
        lce.lce_device_status_reset()
    assert lce.lce_device_status() == 0
    assert np.array_equal(lce.lce_bconv2d(desc, aw, wp).cpu().numpy(), acc)   # still exact afterwards
    lce.lce_plan_run(plan)
    torch.cuda.synchronize()
    assert np.array_equal(plan.out.cpu().numpy(), acc)
    lce.lce_plan_destroy(plan)
    assert lce.lce_device_status() == 0


def test_wait_probe_rejects_limits_outside_its_range():
    for bad in (0, 2_000_000_000):
        with pytest.raises(lce.LceError) as e:
            lce.lce_device_wait_probe(bad)
        assert e.value.status == 1
