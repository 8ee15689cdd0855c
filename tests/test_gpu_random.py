"""GPU parity: dropit_compress_random against the oracle's random strategy (Sec. 3.3 "Random Elements"), bit-exact."""
import numpy as np
import pytest
import torch

import dropit_inputs as di
import oracle
import paper_2202_13808_b200 as dropit
from _parity import assert_cache_matches_oracle, np_bits

pytestmark = pytest.mark.gpu

CASES = [
    (di.small_linear(1, 1, 1, "bf16", 0.5), 0), (di.small_linear(1, 7, 1, "bf16", 0.5), 1),
    (di.small_linear(3, 11, 1, "f32", 0.9), 2), (di.small_linear(37, 129, 1, "bf16", 0.9), 3),
    (di.small_linear(64, 768, 1, "f32", 0.9), 2 ** 63 + 5), (di.small_linear(1031, 769, 1, "bf16", 0.9), 0xFFFFFFFFFFFFFFFF),
    (di.small_linear(1031, 769, 1, "f32", 0.8), 7), (di.small_linear(512, 768, 1, "bf16", 0.0), 8),
    (di.small_linear(512, 768, 1, "bf16", 1.0), 9), (di.small_linear(1, (1 << 19) + 519, 1, "bf16", 0.5), 10),
    (di.small_conv(4, 64, 56, 56, 1, 1, 1, gamma=0.8), 11),
]


@pytest.mark.parametrize("fmt", ["bitmask", "index32"])
@pytest.mark.parametrize("case,seed", CASES, ids=lambda c: getattr(c, "name", str(c)))
def test_random_compress_matches_oracle(cuda_device, case, seed, fmt):
    x = di.make_x(case)
    bits, dt = oracle.to_bits(x)
    keep, k = oracle.random_k(bits.size, case.gamma, seed)
    cache = dropit.dropit_compress_random(x.to(cuda_device), case.gamma, seed, fmt)
    dropit.check_device_status(cuda_device)
    assert_cache_matches_oracle(cache, bits, dt, keep, k, fmt)
    rec = dropit.dropit_decompress(cache)
    assert (np_bits(rec) == np.where(keep == 1, bits, 0).astype(bits.dtype)).all()


def test_full_size_and_weight_grad_from_a_random_cache(cuda_device):
    case = di.VITB_FC1
    x, dy = di.make_x(case), di.make_dy(case)
    bits, dt = oracle.to_bits(x)
    keep, k = oracle.random_k(bits.size, case.gamma, 123)
    cache = dropit.dropit_compress_random(x.to(cuda_device), case.gamma, 123)
    dropit.check_device_status(cuda_device)
    assert_cache_matches_oracle(cache, bits, dt, keep, k, "bitmask")
    dw = dropit.dropit_weight_grad(dy.to(cuda_device), cache).cpu().numpy()
    dyb, _ = oracle.to_bits(dy)
    rng = np.random.default_rng(0)
    js, cs = rng.integers(0, case.Cz, 200), rng.integers(0, case.Ca, 200)
    ref = oracle.fc_weight_grad_entries(dyb, bits, keep, case.M, case.Ca, case.Cz, dt, js, cs)
    scale = np.abs(ref).max()
    assert np.abs(dw[js, cs] - ref).max() / scale < 1e-2      # bf16 inputs, fp32 accumulation


def test_same_seed_same_mask_whatever_the_data(cuda_device):
    a = torch.randn(300, 512, device=cuda_device, dtype=torch.bfloat16)
    b = torch.randn(300, 512, device=cuda_device, dtype=torch.float32)
    ca, cb = dropit.dropit_compress_random(a, 0.9, 5), dropit.dropit_compress_random(b, 0.9, 5)
    cc = dropit.dropit_compress_random(a, 0.9, 6)
    assert torch.equal(ca.meta, cb.meta) and torch.equal(ca.offsets, cb.offsets)
    assert not torch.equal(ca.meta, cc.meta)


def test_random_layer_trains_and_draws_a_new_mask_per_call(cuda_device):
    torch.manual_seed(0)
    lin = dropit.DropITLinear(256, 128, gamma=0.5, strategy="random", seed=3, device=cuda_device, dtype=torch.bfloat16)
    x = torch.randn(64, 256, device=cuda_device, dtype=torch.bfloat16, requires_grad=True)
    lin(x).float().sum().backward()
    first = lin.weight.grad.clone()
    lin.weight.grad = None
    lin(x).float().sum().backward()                      # the seed advances: another mask
    assert not torch.equal(first, lin.weight.grad)
    # the random estimate is (1 - gamma) times the dense gradient in expectation (App. A.3 with a random mask)
    dense = torch.ones(64, 128, device=cuda_device).t() @ x.detach().float()
    ratio = (first.float() * dense).sum() / (dense * dense).sum()
    assert 0.4 < float(ratio) < 0.6
