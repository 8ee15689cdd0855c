"""GPU parity: dropit_compress / dropit_decompress against the CPU oracle, bit-exact."""
import numpy as np
import pytest
import torch

import dropit_inputs as di
import oracle
import paper_2202_13808_b200 as dropit
from _parity import assert_cache_matches_oracle, np_bits, oracle_cache

pytestmark = pytest.mark.gpu

SMALL = [
    di.small_linear(1, 1, 1, "bf16", 0.0), di.small_linear(1, 1, 1, "bf16", 0.5), di.small_linear(1, 7, 1, "bf16", 0.5),
    di.small_linear(3, 11, 1, "bf16", 0.9), di.small_linear(1, 127, 1, "bf16", 0.9), di.small_linear(1, 129, 1, "f32", 0.9),
    di.small_linear(37, 129, 1, "bf16", 0.9), di.small_linear(64, 768, 1, "bf16", 0.9), di.small_linear(64, 768, 1, "f32", 0.9),
    di.small_linear(256, 768, 1, "f32", 0.9),                        # the single-Linear fp32 case
    di.small_linear(1031, 769, 1, "bf16", 0.9),                      # several tiles + ragged tail
    di.small_linear(1031, 769, 1, "f32", 0.8),
    di.small_linear(300, 3072, 1, "bf16", 0.9, "gelu"),
    di.small_linear(512, 768, 1, "bf16", 0.5), di.small_linear(512, 768, 1, "bf16", 0.8),
    di.small_linear(512, 768, 1, "bf16", 0.0), di.small_linear(512, 768, 1, "bf16", 1.0),
    di.small_linear(333, 100, 1, "f32", 0.0), di.small_linear(333, 100, 1, "f32", 1.0),
    di.small_conv(4, 64, 56, 56, 1, 1, 1, gamma=0.8),               # ReLU: half exact zeros
    di.small_conv(3, 5, 17, 13, 1, 1, 1, gamma=0.3),                 # threshold falls inside the zero ties
    di.small_conv(3, 5, 17, 13, 1, 1, 1, gamma=0.8, dtype="f32"),
]


@pytest.mark.parametrize("fmt", ["bitmask", "index32"])
@pytest.mark.parametrize("case", SMALL, ids=lambda c: c.name)
def test_compress_matches_oracle_small(cuda_device, case, fmt):
    x = di.make_x(case)
    bits, dt, keep, k = oracle_cache(x, case.gamma)
    cache = dropit.dropit_compress(x.to(cuda_device), case.gamma, fmt)
    dropit.check_device_status(cuda_device)
    assert_cache_matches_oracle(cache, bits, dt, keep, k, fmt)
    # R(a-hat): retained values untouched, dropped positions +0
    rec = dropit.dropit_decompress(cache)
    expect = np.where(keep == 1, bits, 0).astype(bits.dtype)
    assert (np_bits(rec) == expect).all()


def _special(bits_np, torch_dtype, gamma, fmt, dev):
    t = torch.from_numpy(bits_np.view(np.int16 if torch_dtype == torch.bfloat16 else np.int32)).view(torch_dtype)
    dt = oracle.BF16 if torch_dtype == torch.bfloat16 else oracle.F32
    keep, k = oracle.min_k(bits_np, gamma, dt)
    cache = dropit.dropit_compress(t.to(dev), gamma, fmt)
    dropit.check_device_status(dev)
    assert_cache_matches_oracle(cache, bits_np, dt, keep, k, fmt)
    return keep


@pytest.mark.parametrize("fmt", ["bitmask", "index32"])
def test_degenerate_tensors(cuda_device, fmt):
    n = 20011
    # all equal magnitude, alternating sign: the lowest indices win
    x = np.full(n, 0x3F80, np.uint16); x[::2] |= 0x8000
    keep = _special(x, torch.bfloat16, 0.7, fmt, cuda_device)
    k = int(keep.sum()); assert keep[:k].all()
    # all zeros (+0 and -0)
    x = np.zeros(n, np.uint16); x[1::3] = 0x8000
    _special(x, torch.bfloat16, 0.5, fmt, cuda_device)
    # strictly increasing magnitude
    x = (np.arange(1, n + 1, dtype=np.float32) * np.where(np.arange(n) % 2, -1, 1)).astype(np.float32).view(np.uint32)
    keep = _special(x, torch.float32, 0.9, fmt, cuda_device)
    assert keep[-int(keep.sum()):].all()
    # Inf / NaN patterns / denormals / -0 are ordered by raw magnitude bits and stored verbatim
    rng = np.random.default_rng(3)
    x = rng.integers(0, 1 << 16, n).astype(np.uint16)
    _special(x, torch.bfloat16, 0.9, fmt, cuda_device)
    x = rng.integers(0, 1 << 32, n, dtype=np.uint64).astype(np.uint32)
    _special(x, torch.float32, 0.6, fmt, cuda_device)
    # few distinct values: massive ties at the threshold, across many tiles
    x = rng.integers(0, 3, 100003).astype(np.uint16) * 0x0100 + 0x3F00
    _special(x, torch.bfloat16, 0.55, fmt, cuda_device)
    x = (rng.integers(0, 3, 100003).astype(np.uint32) << 23) + 0x3F000000
    _special(x, torch.float32, 0.55, fmt, cuda_device)


# sampled (fast) path with every kind of tail: whole super-blocks, one element more, half a super-block,
# a ragged last vector, one element short of a super-block
TAILS = [1 << 19, (1 << 19) + 1, (1 << 19) + 512, (1 << 19) + 519, (1 << 19) + 1023, (1 << 19) + 1025,
         148 * 32 * 1024 + 8, 148 * 32 * 2048 - 1]


@pytest.mark.parametrize("fmt", ["bitmask", "index32"])
@pytest.mark.parametrize("n", TAILS)
def test_sampled_path_tails(cuda_device, n, fmt):
    case = di.small_linear(1, n, 1, "bf16", 0.9, "gelu" if n % 2 else "normal")
    x = di.make_x(case)
    bits, dt, keep, k = oracle_cache(x, case.gamma)
    cache = dropit.dropit_compress(x.to(cuda_device), case.gamma, fmt)
    dropit.check_device_status(cuda_device)
    assert_cache_matches_oracle(cache, bits, dt, keep, k, fmt)
    rec = dropit.dropit_decompress(cache)
    assert (np_bits(rec) == np.where(keep == 1, bits, 0).astype(bits.dtype)).all()


@pytest.mark.parametrize("fmt", ["bitmask", "index32"])
def test_degenerate_tensors_on_the_sampled_path(cuda_device, fmt):
    """Large tensors (sampled band, per-warp histograms) whose threshold sits in a huge tie."""
    n = (1 << 20) + 777
    rng = np.random.default_rng(11)
    # ReLU-like: half exact zeros, and more elements to retain than there are non-zeros: T = 0, the quota ends among the zeros
    x = np.abs(rng.standard_normal(n)).astype(np.float32)
    x[rng.random(n) < 0.5] = 0.0
    bits = (x.view(np.uint32) >> 16).astype(np.uint16)
    bits[::7] |= 0x8000                                   # some -0 and negative values
    _special(bits, torch.bfloat16, 0.3, fmt, cuda_device)
    # all equal magnitude: the lowest indices win
    x = np.full(n, 0x3F80, np.uint16); x[::2] |= 0x8000
    keep = _special(x, torch.bfloat16, 0.7, fmt, cuda_device)
    k = int(keep.sum()); assert keep[:k].all() and not keep[k:].any()
    # three distinct magnitudes
    x = rng.integers(0, 3, n).astype(np.uint16) * 0x0100 + 0x3F00
    _special(x, torch.bfloat16, 0.55, fmt, cuda_device)
    # a few huge outliers (Inf, NaN patterns) in Gaussian data
    x = (rng.standard_normal(n).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    x[rng.integers(0, n, 50)] = 0x7F80
    x[rng.integers(0, n, 50)] = 0x7FC1
    _special(x, torch.bfloat16, 0.9, fmt, cuda_device)
    _special(x, torch.bfloat16, 0.999, fmt, cuda_device)


def test_workspace_needs_no_initialisation(cuda_device):
    """The scratch may hold anything: all ones, zeros, random bytes, or what an earlier call on another tensor left."""
    big = di.small_linear(700, 768, 1, "bf16", 0.9)       # sampled path
    small = di.small_linear(37, 129, 1, "bf16", 0.5)      # general path
    xb, xs = di.make_x(big).to(cuda_device), di.make_x(small).to(cuda_device)
    ref_b, ref_s = dropit.dropit_compress(xb, 0.9), dropit.dropit_compress(xs, 0.5)
    nbytes = max(dropit.dropit_cache_sizes(c.n, c.gamma, dropit.BF16, dropit.FMT_BITMASK)[3] for c in (big, small))
    ws = torch.empty(nbytes, dtype=torch.uint8, device=cuda_device)
    g = torch.Generator(device="cpu").manual_seed(5)
    fills = [lambda: ws.fill_(0xFF), lambda: ws.zero_(), lambda: ws.copy_(torch.randint(0, 256, (nbytes,), generator=g,
                                                                                         dtype=torch.uint8)),
             lambda: None, lambda: None]
    for fill in fills:
        fill()
        for x, gamma, ref in ((xb, 0.9, ref_b), (xs, 0.5, ref_s), (xb, 0.9, ref_b)):
            c = dropit.dropit_compress(x, gamma, workspace=ws)
            assert torch.equal(c.values.view(torch.int16), ref.values.view(torch.int16))
            assert torch.equal(c.meta, ref.meta) and torch.equal(c.offsets, ref.offsets)
    dropit.check_device_status(cuda_device)


def test_compress_replayed_from_a_captured_graph(cuda_device):
    """The grid barrier counts under a number that the host draws per call; a captured launch replays the same number
    and must still start from a clean word (the last CTA to leave a launch clears it)."""
    case = di.small_linear(700, 768, 1, "bf16", 0.9)      # sampled path: one grid barrier
    x = di.make_x(case)
    bits, dt, keep, k = oracle_cache(x, case.gamma)
    xd = x.to(cuda_device)
    nbytes = dropit.dropit_cache_sizes(case.n, case.gamma, dropit.BF16, dropit.FMT_BITMASK)[3]
    ws = torch.empty(nbytes, dtype=torch.uint8, device=cuda_device)
    side = torch.cuda.Stream(device=cuda_device)
    side.wait_stream(torch.cuda.current_stream(cuda_device))
    with torch.cuda.stream(side):
        dropit.dropit_compress(xd, case.gamma, "bitmask", workspace=ws)   # attributes and the status word exist before capture
    torch.cuda.current_stream(cuda_device).wait_stream(side)
    torch.cuda.synchronize(cuda_device)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        cache = dropit.dropit_compress(xd, case.gamma, "bitmask", workspace=ws)
    for _ in range(4):
        cache.values.zero_(); cache.meta.zero_(); cache.offsets.zero_()
        graph.replay()
        torch.cuda.synchronize(cuda_device)
        dropit.check_device_status(cuda_device)
        assert_cache_matches_oracle(cache, bits, dt, keep, k, "bitmask")
    again = dropit.dropit_compress(xd, case.gamma, "bitmask", workspace=ws)      # an ordinary call on the same workspace
    dropit.check_device_status(cuda_device)
    assert_cache_matches_oracle(again, bits, dt, keep, k, "bitmask")


def test_decompress_into_a_given_buffer(cuda_device):
    case = di.small_linear(300, 3072, 1, "bf16", 0.9, "gelu")
    x = di.make_x(case).to(cuda_device)
    cache = dropit.dropit_compress(x, case.gamma)
    out = torch.full((case.n,), float("nan"), dtype=torch.bfloat16, device=cuda_device)
    got = dropit.dropit_decompress(cache, out=out)
    assert got.data_ptr() == out.data_ptr()
    assert torch.equal(out.view(torch.int16), dropit.dropit_decompress(cache).reshape(-1).view(torch.int16))
    with pytest.raises(ValueError):
        dropit.dropit_decompress(cache, out=torch.empty(case.n - 1, dtype=torch.bfloat16, device=cuda_device))
    with pytest.raises(ValueError):
        dropit.dropit_decompress(cache, out=torch.empty(case.n, dtype=torch.float32, device=cuda_device))


def test_empty_tensor_is_a_noop(cuda_device):
    cache = dropit.dropit_compress(torch.empty(0, dtype=torch.bfloat16, device=cuda_device), 0.5)
    assert cache.k == 0 and cache.values.numel() == 0 and cache.meta.numel() == 0
    assert dropit.dropit_decompress(cache).numel() == 0


def test_repeat_calls_are_bit_identical(cuda_device):
    case = di.small_linear(2000, 768, 1, "bf16", 0.9)
    x = di.make_x(case).to(cuda_device)
    a = dropit.dropit_compress(x, 0.9)
    for _ in range(3):
        b = dropit.dropit_compress(x, 0.9)
        assert torch.equal(a.values.view(torch.int16), b.values.view(torch.int16))
        assert torch.equal(a.meta, b.meta) and torch.equal(a.offsets, b.offsets)
    dropit.check_device_status(cuda_device)


FULL = [di.VITB_FC1, di.VITB_FC2, di.R50_CONV1X1, di.R50_CONV3X3,
        di.with_gamma(di.VITDET_QKV, 0.5), di.with_gamma(di.VITDET_QKV, 0.8), di.VITDET_QKV,
        di.with_gamma(di.VITDET_FC2, 0.5), di.with_gamma(di.VITDET_FC2, 0.8), di.VITDET_FC2]


@pytest.mark.parametrize("case", FULL, ids=lambda c: c.name)
def test_compress_matches_oracle_full_size(cuda_device, case):
    x = di.make_x(case)
    bits, dt, keep, k = oracle_cache(x, case.gamma)
    xg = x.to(cuda_device)
    cache = dropit.dropit_compress(xg, case.gamma, "bitmask")
    dropit.check_device_status(cuda_device)
    assert_cache_matches_oracle(cache, bits, dt, keep, k, "bitmask")
    rec = dropit.dropit_decompress(cache)
    assert (np_bits(rec) == np.where(keep == 1, bits, 0).astype(bits.dtype)).all()
    if case.n <= 40_000_000:
        cache_i = dropit.dropit_compress(xg, case.gamma, "index32")
        dropit.check_device_status(cuda_device)
        assert_cache_matches_oracle(cache_i, bits, dt, keep, k, "index32")
