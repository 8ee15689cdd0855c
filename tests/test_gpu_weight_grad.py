"""GPU parity: dropit_weight_grad (Eq. 6) against the CPU oracle."""
import numpy as np
import pytest
import torch

import dropit_inputs as di
import oracle
import paper_2202_13808_b200 as dropit
from _parity import max_rel_err, oracle_cache

pytestmark = pytest.mark.gpu

TOL = {"bf16": 1e-2, "f32": 1e-5}          # max-norm relative error, bf16 inputs / fp32 inputs
TIGHT = {"bf16": 2e-4, "f32": 1e-5}        # what fp32 accumulation of exact products should reach

SMALL = [
    di.small_linear(256, 768, 768, "f32", 0.9, dy_std=1.0),           # the single-Linear fp32 configuration
    di.small_linear(64, 128, 256, "bf16", 0.9),
    di.small_linear(640, 768, 384, "bf16", 0.9),                       # several k-blocks, 3 column tiles
    di.small_linear(1000, 512, 384, "bf16", 0.9),                      # ragged token count (1000 = 15*64 + 40)
    di.small_linear(200, 264, 136, "bf16", 0.5),                       # ragged tiles in both output dims
    di.small_linear(200, 100, 36, "bf16", 0.5),                        # widths the TMA path cannot take
    di.small_linear(129, 65, 33, "f32", 0.5, dy_std=1.0),
    di.small_linear(300, 3072, 128, "bf16", 0.9, "gelu"),
    di.small_linear(512, 256, 128, "bf16", 0.0),                       # gamma = 0: the dense gradient
    di.small_linear(512, 256, 128, "bf16", 1.0),                       # gamma = 1: zero gradient
    di.small_linear(8192, 256, 128, "bf16", 0.9),                      # one tile, deep split along tokens
    di.small_linear(200, 2056, 1000, "bf16", 0.9),                     # 72 tiles x 2 splits, ragged tiles
    di.small_linear(512, 1792, 520, "bf16", 0.9),                      # 35 tiles (42 in CTA pairs: a pair half past the last row), ragged rows
    # the scratch is produced inside the GEMM kernel (channel counts that are multiples of 64):
    di.small_linear(131, 192, 64, "bf16", 0.7),                        # ragged last step (n = 24 * 1024 + 576), ragged k-block
    di.small_linear(333, 320, 192, "bf16", 0.5),                       # two column tiles, the second one partial
    di.small_linear(700, 256, 256, "bf16", 0.2),                       # dense steps: more values than the look-ahead window
    di.small_linear(4100, 1024, 1152, "bf16", 0.9),                    # 36 tiles (40 in CTA pairs) x 4 / 3 splits
    di.small_linear(2000, 2048, 1152, "bf16", 0.8),                    # 72 tiles x 2 splits
    di.small_linear(1500, 1280, 384, "bf16", 0.9),                     # 15 tiles x 9 splits (20 x 7 in CTA pairs): eight parts per tile
    di.small_linear(300, 256, 256, "bf16", 0.5),                       # half of every row retained: runs longer than the value window
    di.small_linear(777, 384, 200, "bf16", 0.6),                       # ragged tokens and outputs, dense rows
    di.small_linear(4096, 128, 8, "bf16", 0.95),                       # one channel tile, eight outputs
]


def _run(case, fmt, dev):
    x, dy = di.make_x(case), di.make_dy(case)
    bits, dt, keep, k = oracle_cache(x, case.gamma)
    dyb, _ = oracle.to_bits(dy)
    cache = dropit.dropit_compress(x.to(dev), case.gamma, fmt)
    dw = dropit.dropit_weight_grad(dy.to(dev), cache)
    dropit.check_device_status(dev)
    return bits, dyb, dt, keep, cache, dw


@pytest.mark.parametrize("fmt", ["bitmask", "index32"])
@pytest.mark.parametrize("case", SMALL, ids=lambda c: c.name)
def test_weight_grad_matches_oracle(cuda_device, case, fmt):
    bits, dyb, dt, keep, cache, dw = _run(case, fmt, cuda_device)
    ref = oracle.fc_weight_grad(dyb, bits, keep, case.M, case.Ca, case.Cz, dt)
    got = dw.cpu().numpy()
    assert got.shape == (case.Cz, case.Ca)
    err = max_rel_err(got, ref)
    assert err <= TOL[case.dtype], err
    assert err <= TIGHT[case.dtype], err
    if case.gamma == 1.0:
        assert not got.any()


# The kernel with one CTA per tile (taken for Cz <= 128, or on request): 2 or 4 splits add up inside a cluster,
# other counts through global memory.
ONE_CTA = [c for c in SMALL if c.dtype == "bf16" and c.Cz > 128 and c.Ca % 8 == 0 and c.Cz % 8 == 0 and c.M >= 200]


@pytest.mark.parametrize("case", ONE_CTA, ids=lambda c: c.name)
def test_weight_grad_one_cta_per_tile_matches_oracle(cuda_device, case, monkeypatch):
    monkeypatch.setenv("DROPIT_WG_PATH", "single")
    bits, dyb, dt, keep, cache, dw = _run(case, "bitmask", cuda_device)
    ref = oracle.fc_weight_grad(dyb, bits, keep, case.M, case.Ca, case.Cz, dt)
    assert max_rel_err(dw.cpu().numpy(), ref) <= TIGHT[case.dtype]


FUSED = [c for c in SMALL if c.dtype == "bf16" and c.Ca % 128 == 0 and c.Cz % 8 == 0] + [
    di.small_linear(1000, 384, 520, "bf16", 0.9),          # ragged rows of the 256-row tile, 128-channel tail tile
    di.small_linear(700, 256, 256, "bf16", 0.3),           # dense rows: more retained values than the prefetched window
    di.small_linear(130, 128, 64, "bf16", 0.0),
]


@pytest.mark.parametrize("case", FUSED, ids=lambda c: c.name)
def test_fused_weight_grad_matches_oracle(cuda_device, case):
    """dropit_weight_grad_fused: the cache is expanded inside the GEMM, no dense scratch."""
    x, dy = di.make_x(case), di.make_dy(case)
    bits, dt, keep, k = oracle_cache(x, case.gamma)
    dyb, _ = oracle.to_bits(dy)
    cache = dropit.dropit_compress(x.to(cuda_device), case.gamma, "bitmask")
    dw = dropit.dropit_weight_grad(dy.to(cuda_device), cache, fused=True)
    dropit.check_device_status(cuda_device)
    ref = oracle.fc_weight_grad(dyb, bits, keep, case.M, case.Ca, case.Cz, dt)
    err = max_rel_err(dw.cpu().numpy(), ref)
    assert err <= TOL["bf16"] and err <= TIGHT["bf16"], err
    # both variants add the same exact bf16 products in fp32; they agree to rounding of the split order
    dw2 = dropit.dropit_weight_grad(dy.to(cuda_device), cache)
    assert torch.allclose(dw, dw2, rtol=1e-4, atol=1e-6 * float(dw2.abs().max()))
    # reproducible run to run
    assert torch.equal(dw, dropit.dropit_weight_grad(dy.to(cuda_device), cache, fused=True))
    # accumulate adds to what is there
    out = torch.full_like(dw, 0.25)
    dropit.dropit_weight_grad(dy.to(cuda_device), cache, out=out, accumulate=True, fused=True)
    assert torch.allclose(out, dw + 0.25, rtol=1e-6, atol=1e-6)


def test_fused_weight_grad_full_size_and_unsupported(cuda_device):
    case = di.VITB_FC2
    bits, dyb, dt, keep, cache, dw = _run(case, "bitmask", cuda_device)
    dwf = dropit.dropit_weight_grad(di.make_dy(case).to(cuda_device), cache, fused=True)
    dropit.check_device_status(cuda_device)
    assert torch.allclose(dwf, dw, rtol=1e-4, atol=1e-6 * float(dw.abs().max()))
    rng = np.random.default_rng(1)
    js, cs = rng.integers(0, case.Cz, 2000), rng.integers(0, case.Ca, 2000)
    ref = oracle.fc_weight_grad_entries(dyb, bits, keep, case.M, case.Ca, case.Cz, dt, js, cs)
    err = np.abs(dwf.cpu().numpy()[js, cs] - ref).max() / np.abs(ref).max()
    assert err <= TIGHT["bf16"], err
    small = di.small_linear(64, 100, 36, "bf16", 0.5)
    c2 = dropit.dropit_compress(di.make_x(small).to(cuda_device), 0.5, "bitmask")
    with pytest.raises(dropit.DropITError):
        dropit.dropit_weight_grad(di.make_dy(small).to(cuda_device), c2, fused=True)


@pytest.mark.parametrize("case", [di.small_linear(640, 768, 384, "bf16", 0.9),       # partial planes in global memory
                                  di.small_linear(200, 2056, 1000, "bf16", 0.9)],    # cluster exchange
                         ids=lambda c: c.name)
def test_accumulate_adds_to_existing_gradient(cuda_device, case):
    bits, dyb, dt, keep, cache, dw = _run(case, "bitmask", cuda_device)
    base = torch.full_like(dw, 0.5)
    out = base.clone()
    dropit.dropit_weight_grad(di.make_dy(case).to(cuda_device), cache, out=out, accumulate=True)
    assert torch.allclose(out, dw + base, rtol=1e-6, atol=1e-6)
    out2 = torch.full_like(dw, 7.0)
    dropit.dropit_weight_grad(di.make_dy(case).to(cuda_device), cache, out=out2, accumulate=False)
    assert torch.equal(out2, dw)


def test_weight_grad_scratch_needs_no_initialisation(cuda_device):
    """The workspace (split counters, ready flags of the in-kernel production, dense scratch) may hold
    anything: bytes of one value, random bytes, or what an earlier call on another tensor left there."""
    case = di.small_linear(2000, 2048, 1152, "bf16", 0.8)
    bits, dyb, dt, keep, cache, dw = _run(case, "bitmask", cuda_device)
    dy = di.make_dy(case).to(cuda_device)
    wb = dropit.dropit_weight_grad_workspace(case.M, case.Ca, case.Cz, dropit.BF16, dropit.FMT_BITMASK, cuda_device)
    g = torch.Generator(device="cpu").manual_seed(5)
    fills = [torch.zeros(wb, dtype=torch.uint8), torch.full((wb,), 0xFF, dtype=torch.uint8),
             torch.randint(0, 256, (wb,), dtype=torch.uint8, generator=g)]
    for f in fills:
        ws = f.to(cuda_device)
        for _ in range(2):     # the second call finds the first call's flags
            out = dropit.dropit_weight_grad(dy, cache, workspace=ws)
            dropit.check_device_status(cuda_device)
            assert torch.equal(out, dw)
    other = di.small_linear(1000, 2048, 1152, "bf16", 0.5)
    c2 = dropit.dropit_compress(di.make_x(other).to(cuda_device), other.gamma, "bitmask")
    ws = torch.empty(wb, dtype=torch.uint8, device=cuda_device)
    dropit.dropit_weight_grad(di.make_dy(other).to(cuda_device), c2, workspace=ws)
    assert torch.equal(dropit.dropit_weight_grad(dy, cache, workspace=ws), dw)
    dropit.check_device_status(cuda_device)


def test_weight_grad_is_reproducible(cuda_device):
    case = di.small_linear(8192, 256, 128, "bf16", 0.9)
    bits, dyb, dt, keep, cache, dw = _run(case, "bitmask", cuda_device)
    dy = di.make_dy(case).to(cuda_device)
    for _ in range(3):
        assert torch.equal(dropit.dropit_weight_grad(dy, cache), dw)


def test_weight_grad_replayed_from_a_captured_graph(cuda_device):
    """The tile counters of the split reduction carry a number that the host draws per call; a captured launch
    replays the same number, and still has to start from clean counts (the finisher of a part clears them)."""
    case = di.small_linear(2000, 2048, 1152, "bf16", 0.8)      # two splits per tile
    bits, dyb, dt, keep, cache, dw = _run(case, "bitmask", cuda_device)
    dy = di.make_dy(case).to(cuda_device)
    wb = dropit.dropit_weight_grad_workspace(case.M, case.Ca, case.Cz, 0, 0, cuda_device)
    ws = torch.empty(wb, dtype=torch.uint8, device=cuda_device)
    out = torch.empty_like(dw)
    side = torch.cuda.Stream(device=cuda_device)
    side.wait_stream(torch.cuda.current_stream(cuda_device))
    with torch.cuda.stream(side):
        dropit.dropit_weight_grad(dy, cache, out=out, workspace=ws)      # attributes and the status word exist before capture
    torch.cuda.current_stream(cuda_device).wait_stream(side)
    torch.cuda.synchronize(cuda_device)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        dropit.dropit_weight_grad(dy, cache, out=out, workspace=ws)
    for _ in range(3):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize(cuda_device)
        dropit.check_device_status(cuda_device)
        assert torch.equal(out, dw)
    assert torch.equal(dropit.dropit_weight_grad(dy, cache, workspace=ws), dw)   # an ordinary call on the same workspace


FULL_SIZE = [di.VITB_FC1, di.VITB_FC2,
             di.with_gamma(di.VITDET_QKV, 0.5), di.with_gamma(di.VITDET_QKV, 0.8), di.VITDET_QKV,
             di.with_gamma(di.VITDET_FC1, 0.5), di.VITDET_FC1,
             di.with_gamma(di.VITDET_FC2, 0.5), di.VITDET_FC2]


@pytest.mark.parametrize("case", FULL_SIZE, ids=lambda c: c.name)
def test_weight_grad_full_size_sampled_entries(cuda_device, case):
    bits, dyb, dt, keep, cache, dw = _run(case, "bitmask", cuda_device)
    got = dw.cpu().numpy()
    rng = np.random.default_rng(0)
    js = np.concatenate([rng.integers(0, case.Cz, 3000), [0, case.Cz - 1, 0, case.Cz - 1, 127, 128]])
    cs = np.concatenate([rng.integers(0, case.Ca, 3000), [0, 0, case.Ca - 1, case.Ca - 1, 255, 256]])
    ref = oracle.fc_weight_grad_entries(dyb, bits, keep, case.M, case.Ca, case.Cz, dt, js, cs)
    err = np.abs(got[js, cs] - ref).max() / np.abs(ref).max()
    assert err <= TOL["bf16"] and err <= TIGHT["bf16"], err
    # a property that holds at any size: column c of dW is zero iff no element of column c was retained
    col_kept = keep.reshape(case.M, case.Ca).any(axis=0)
    assert (np.abs(got).max(axis=0)[~col_kept] == 0).all()
