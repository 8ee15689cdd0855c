"""The bounded device-side waits give up and report it, instead of hanging.

Every wait inside the kernels (grid barrier of the selection kernel, pipeline barriers of the weight-gradient
kernels) counts its polls against a limit.  DROPIT_TEST_SPIN_LIMIT (read by the library at every call)
shrinks that limit to a handful of polls, so that on a large tensor the waits run out long before the data
arrives.  What must hold then: the call returns, the status word says DROPIT_ERR_TIMEOUT (or, if no wait
happened to run out, the result is still exact), and the next ordinary call is exact again.  Nothing here
faults or hangs the device: a wait that gives up makes its kernel skip the remaining work and return.
"""
import numpy as np
import pytest
import torch

import dropit_inputs as di
import oracle
import paper_2202_13808_b200 as dropit
from _parity import assert_cache_matches_oracle, max_rel_err, oracle_cache

pytestmark = pytest.mark.gpu

ERR_TIMEOUT = 5


def _status_after_sync(dev):
    """None if the device status word is clean, else the code it held (the word is cleared)."""
    try:
        dropit.check_device_status(dev)
    except dropit.DropITError as e:
        return e.code
    return None


def test_compress_grid_barrier_gives_up_and_recovers(cuda_device, monkeypatch):
    case = di.VITB_FC1
    x = di.make_x(case)
    bits, dt, keep, k = oracle_cache(x, case.gamma)
    xd = x.to(cuda_device)
    monkeypatch.setenv("DROPIT_TEST_SPIN_LIMIT", "2")
    timed_out = 0
    for _ in range(3):
        cache = dropit.dropit_compress(xd, case.gamma, "bitmask")     # must return
        code = _status_after_sync(cuda_device)
        assert code in (None, ERR_TIMEOUT)
        if code is None:
            assert_cache_matches_oracle(cache, bits, dt, keep, k, "bitmask")
        else:
            timed_out += 1
    monkeypatch.delenv("DROPIT_TEST_SPIN_LIMIT")
    cache = dropit.dropit_compress(xd, case.gamma, "bitmask")
    assert _status_after_sync(cuda_device) is None
    assert_cache_matches_oracle(cache, bits, dt, keep, k, "bitmask")
    # 148 CTAs that give up after two polls of a barrier which takes microseconds to fill: the limit bites
    assert timed_out >= 1


@pytest.mark.parametrize("path", ["scratch", "fused"])
def test_weight_grad_pipeline_waits_give_up_and_recover(cuda_device, monkeypatch, path):
    if path == "fused":     # the kernel that expands the cache into tensor memory, taken by the ordinary entry point
        monkeypatch.setenv("DROPIT_WG_PATH", "fused")
    case = di.small_linear(4100, 1024, 1152, "bf16", 0.9)
    x, dy = di.make_x(case), di.make_dy(case)
    bits, dt, keep, k = oracle_cache(x, case.gamma)
    dyb, _ = oracle.to_bits(dy)
    ref = oracle.fc_weight_grad(dyb, bits, keep, case.M, case.Ca, case.Cz, dt)
    cache = dropit.dropit_compress(x.to(cuda_device), case.gamma, "bitmask")
    dyd = dy.to(cuda_device)
    good = dropit.dropit_weight_grad(dyd, cache)
    assert _status_after_sync(cuda_device) is None
    assert max_rel_err(good.cpu().numpy(), ref) <= 2e-4
    monkeypatch.setenv("DROPIT_TEST_SPIN_LIMIT", "1")
    timed_out = 0
    for _ in range(3):
        out = dropit.dropit_weight_grad(dyd, cache)                   # must return
        code = _status_after_sync(cuda_device)
        assert code in (None, ERR_TIMEOUT)
        if code is None:
            assert torch.equal(out, good)
        else:
            timed_out += 1
    monkeypatch.delenv("DROPIT_TEST_SPIN_LIMIT")
    again = dropit.dropit_weight_grad(dyd, cache)
    assert _status_after_sync(cuda_device) is None
    assert torch.equal(again, good)
    assert timed_out >= 1
