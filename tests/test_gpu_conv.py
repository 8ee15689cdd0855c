"""GPU parity: dropit_conv_weight_grad (Eq. 4-5) against the CPU oracle."""
import numpy as np
import pytest
import torch

import dropit_inputs as di
import oracle
import paper_2202_13808_b200 as dropit
from _parity import max_rel_err, oracle_cache

pytestmark = pytest.mark.gpu

TOL = {"bf16": 1e-2, "f32": 1e-5}
TIGHT = {"bf16": 2e-4, "f32": 1e-5}

SMALL = [
    di.small_conv(2, 16, 14, 14, 32, 1, 1, 1, 0, "bf16", 0.8),
    di.small_conv(2, 16, 14, 14, 32, 3, 3, 1, 1, "bf16", 0.8),
    di.small_conv(3, 5, 9, 7, 4, 3, 3, 1, 1, "bf16", 0.5),           # ragged channels and image
    di.small_conv(3, 5, 9, 8, 4, 3, 3, 2, 1, "f32", 0.5),            # stride 2
    di.small_conv(2, 3, 12, 12, 6, 5, 5, 1, 2, "f32", 0.8),          # 25 taps: more than one sweep
    di.small_conv(2, 8, 10, 10, 8, 3, 2, 1, 0, "bf16", 0.0),         # gamma = 0, no padding, non-square filter
    di.small_conv(2, 8, 10, 10, 8, 3, 3, 1, 1, "bf16", 1.0),         # gamma = 1
    di.small_conv(70, 8, 6, 6, 8, 3, 3, 1, 1, "bf16", 0.8),          # more images than splits
    # shapes the tensor-core path takes (bf16, stride 1, rows a multiple of 8 pixels)
    di.small_conv(2, 16, 16, 16, 32, 3, 3, 1, 1, "bf16", 0.8),       # k-block = 4 rows x 16 pixels
    di.small_conv(2, 24, 8, 8, 40, 3, 3, 1, 1, "bf16", 0.8),         # k-block = 8 x 8, three taps stacked in N
    di.small_conv(3, 130, 24, 32, 200, 3, 3, 1, 1, "bf16", 0.8),     # two row tiles, ragged channel tile
    di.small_conv(2, 300, 16, 16, 20, 1, 1, 1, 0, "bf16", 0.8),      # 1x1: flattened plane, two channel tiles
    di.small_conv(2, 8, 16, 24, 8, 5, 5, 1, 2, "bf16", 0.5),         # 25 taps, five stacked
    di.small_conv(2, 8, 12, 16, 8, 3, 1, 1, 0, "bf16", 0.8),         # no padding: Ho < H
    di.small_conv(1, 16, 4, 72, 16, 3, 3, 1, 1, "bf16", 0.8),        # rows wider than one k-block
    di.small_conv(2, 3, 16, 16, 8, 7, 7, 1, 3, "bf16", 0.5),         # 7x7 on 3 channels
    di.small_conv(150, 8, 8, 8, 8, 3, 3, 1, 1, "bf16", 0.8),         # more k-blocks than splits, uneven
    di.small_conv(4, 256, 14, 14, 256, 3, 3, 1, 1, "bf16", 0.8),     # ResNet stage-3 shape: rows padded to 16 pixels
    di.small_conv(4, 512, 7, 7, 128, 1, 1, 1, 0, "bf16", 0.8),       # 7x7 planes flattened to 49 -> 56 pixels
    di.small_conv(2, 24, 11, 13, 24, 5, 3, 1, 1, "bf16", 0.5),       # Ho != H, Wo = W, odd sizes, non-square filter
    di.small_conv(2, 16, 16, 16, 24, 3, 3, 2, 1, "bf16", 0.8),       # stride 2: one pre-sampled copy per tap
    di.small_conv(2, 8, 15, 15, 8, 1, 1, 2, 0, "bf16", 0.8),         # 1x1 stride 2 (shortcut), odd image
    di.small_conv(1, 3, 32, 32, 16, 7, 7, 2, 3, "bf16", 0.5),        # 7x7 stride 2 pad 3 on 3 channels (stem)
    di.small_conv(2, 130, 28, 28, 140, 3, 3, 2, 1, "bf16", 0.8),     # stride 2, two row tiles, ragged channels
    di.small_conv(4, 64, 56, 56, 64, 3, 3, 1, 1, "bf16", 0.8),       # the ResNet stage-1 3x3 shape, 4 images
    di.small_conv(4, 256, 56, 56, 64, 1, 1, 1, 0, "bf16", 0.8),      # the ResNet stage-1 1x1 shape, 4 images
]


def _run(case, fmt, dev):
    x, dy = di.make_x(case), di.make_dy(case)
    bits, dt, keep, k = oracle_cache(x, case.gamma)
    dyb, _ = oracle.to_bits(dy)
    cache = dropit.dropit_compress(x.to(dev), case.gamma, fmt)
    dw = dropit.dropit_conv_weight_grad(dy.to(dev), cache, (case.R, case.S), case.stride, case.pad)
    dropit.check_device_status(dev)
    return bits, dyb, dt, keep, cache, dw


@pytest.mark.parametrize("fmt", ["bitmask", "index32"])
@pytest.mark.parametrize("case", SMALL, ids=lambda c: c.name)
def test_conv_weight_grad_matches_oracle(cuda_device, case, fmt):
    bits, dyb, dt, keep, cache, dw = _run(case, fmt, cuda_device)
    got = dw.cpu().numpy()
    assert got.shape == (case.Cz, case.Ca, case.R, case.S)
    if case.n * case.Cz * case.R * case.S <= 2e9:
        ref = oracle.conv_weight_grad(dyb, bits, keep, case.B, case.Ca, case.H, case.W, case.Cz, case.R, case.S,
                                      case.stride, case.pad, dt)
        err = max_rel_err(got, ref)
    else:
        rng = np.random.default_rng(1)
        ns = 1500
        js, cs = rng.integers(0, case.Cz, ns), rng.integers(0, case.Ca, ns)
        us, vs = rng.integers(0, case.R, ns), rng.integers(0, case.S, ns)
        ref = oracle.conv_weight_grad_entries(dyb, bits, keep, case.B, case.Ca, case.H, case.W, case.Cz, case.R, case.S,
                                              case.stride, case.pad, dt, js, cs, us, vs)
        err = np.abs(got[js, cs, us, vs] - ref).max() / np.abs(ref).max()
    assert err <= TOL[case.dtype] and err <= TIGHT[case.dtype], err
    if case.gamma == 1.0:
        assert not got.any()


@pytest.mark.parametrize("case", [di.R50_CONV1X1, di.R50_CONV3X3], ids=lambda c: c.name)
def test_conv_full_size_sampled_entries(cuda_device, case):
    bits, dyb, dt, keep, cache, dw = _run(case, "bitmask", cuda_device)
    got = dw.cpu().numpy()
    rng = np.random.default_rng(2)
    ns = 400
    js, cs = rng.integers(0, case.Cz, ns), rng.integers(0, case.Ca, ns)
    us, vs = rng.integers(0, case.R, ns), rng.integers(0, case.S, ns)
    ref = oracle.conv_weight_grad_entries(dyb, bits, keep, case.B, case.Ca, case.H, case.W, case.Cz, case.R, case.S,
                                          case.stride, case.pad, dt, js, cs, us, vs)
    err = np.abs(got[js, cs, us, vs] - ref).max() / np.abs(ref).max()
    assert err <= TOL["bf16"] and err <= TIGHT["bf16"], err


def test_conv_accumulate(cuda_device):
    case = di.small_conv(2, 16, 14, 14, 32, 3, 3, 1, 1, "bf16", 0.8)
    bits, dyb, dt, keep, cache, dw = _run(case, "bitmask", cuda_device)
    out = torch.full_like(dw, 0.25)
    dropit.dropit_conv_weight_grad(di.make_dy(case).to(cuda_device), cache, (3, 3), 1, 1, out=out, accumulate=True)
    assert torch.allclose(out, dw + 0.25, rtol=1e-6, atol=1e-6)
