"""GPU parity for the producer in front of the path (Sec. 3.5): the activation tables, y = act(x), and the cache
that dropit_compress_prepared builds from the producer's statistics, each against the CPU oracle on the same
seeded inputs; everything is bit-exact (the tables are correctly rounded on both sides)."""
import numpy as np
import pytest
import torch

import dropit_inputs as di
import oracle
import paper_2202_13808_b200 as dropit
from _parity import assert_cache_matches_oracle, np_bits

pytestmark = pytest.mark.gpu

KINDS = {"identity": oracle.ACT_IDENTITY, "relu": oracle.ACT_RELU, "gelu": oracle.ACT_GELU}


@pytest.mark.parametrize("kind", sorted(KINDS))
def test_activation_tables_match_the_oracle_on_every_bit_pattern(cuda_device, kind):
    got = dropit.dropit_activation_table(kind, cuda_device).cpu().numpy().view(np.uint16)
    exp = oracle.activation_table(KINDS[kind])
    bad = np.flatnonzero(got != exp)
    assert bad.size == 0, [(hex(int(b)), hex(int(got[b])), hex(int(exp[b]))) for b in bad[:8]]


def _pre_activation(case, scale=1.0, seed=0):
    """A pre-activation tensor: N(0, scale^2) in bf16 (what a Linear / conv / norm layer hands to its activation)."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    return (torch.randn(case.n, generator=g) * scale).to(torch.bfloat16)


CASES = [
    (di.small_linear(3000, 768, 1, "bf16", 0.9), "gelu", 1.0),            # sampled band, several super-blocks per warp
    (di.small_linear(3000, 768, 1, "bf16", 0.9), "relu", 1.0),            # half the tensor is an exact-zero tie
    (di.small_linear(3000, 768, 1, "bf16", 0.5), "relu", 1.0),            # threshold inside the tie at zero
    (di.small_linear(2999, 771, 1, "bf16", 0.8), "gelu", 1.0),            # ragged length: the last super-block is partial
    (di.small_linear(2999, 771, 1, "bf16", 0.9), "identity", 1.0),
    (di.small_linear(700, 300, 1, "bf16", 0.9), "gelu", 1.0),             # too small to be sampled: no statistics
    (di.small_linear(3000, 768, 1, "bf16", 0.9), "gelu", 40.0),           # many inputs outside the table's shared-memory window
    (di.small_linear(3000, 768, 1, "bf16", 0.9), "gelu", 1e-3),           # ... and below it
    (di.VITB_FC2, "gelu", 1.0),                                           # full size
]


@pytest.mark.parametrize("case,act,scale", CASES, ids=lambda v: getattr(v, "name", str(v)))
@pytest.mark.parametrize("fmt", ["bitmask", "index32"])
def test_produce_then_compress_prepared_matches_oracle(cuda_device, case, act, scale, fmt):
    if case.n > 20_000_000 and fmt == "index32":
        pytest.skip("one format at full size")
    x = _pre_activation(case, scale)
    xb = np_bits(x)
    yb = oracle.apply_table(oracle.activation_table(KINDS[act]), xb)
    keep, k = oracle.min_k(yb, case.gamma, oracle.BF16)
    y, prep = dropit.dropit_produce(x.to(cuda_device), case.gamma, act)
    assert (np_bits(y) == yb).all()
    cache = dropit.dropit_compress_prepared(y, case.gamma, prep, fmt)
    dropit.check_device_status(cuda_device)
    assert_cache_matches_oracle(cache, yb, oracle.BF16, keep, k, fmt)
    # the statistics are only a short cut: the ordinary entry point gives the same cache
    plain = dropit.dropit_compress(y, case.gamma, fmt)
    assert torch.equal(plain.values.view(torch.int16), cache.values.view(torch.int16))
    assert torch.equal(plain.meta, cache.meta) and torch.equal(plain.offsets, cache.offsets)


def test_statistics_that_do_not_fit_the_call_are_ignored(cuda_device):
    case = di.small_linear(3000, 768, 1, "bf16", 0.9)
    x = _pre_activation(case)
    yb = oracle.apply_table(oracle.activation_table(oracle.ACT_GELU), np_bits(x))
    y, prep = dropit.dropit_produce(x.to(cuda_device), 0.9, "gelu")
    for gamma in (0.5, 0.95):                     # statistics taken for another drop ratio
        keep, k = oracle.min_k(yb, gamma, oracle.BF16)
        cache = dropit.dropit_compress_prepared(y, gamma, prep)
        assert_cache_matches_oracle(cache, yb, oracle.BF16, keep, k, "bitmask")
    keep, k = oracle.min_k(yb, 0.9, oracle.BF16)
    # bytes that are no statistics at all (no header): ignored
    garbage = torch.randint(0, 256, (prep.numel(),), dtype=torch.uint8).to(cuda_device)
    cache = dropit.dropit_compress_prepared(y, 0.9, garbage)
    assert_cache_matches_oracle(cache, yb, oracle.BF16, keep, k, "bitmask")
    dropit.check_device_status(cuda_device)


def test_identity_statistics_only_and_argument_errors(cuda_device):
    case = di.small_linear(3000, 768, 1, "bf16", 0.9)
    x = di.make_x(case).to(cuda_device)
    bits, dt = oracle.to_bits(di.make_x(case))
    keep, k = oracle.min_k(bits, 0.9, dt)
    y, prep = dropit.dropit_produce(x, 0.9, "identity", want_y=False)
    assert y is None
    cache = dropit.dropit_compress_prepared(x, 0.9, prep)
    assert_cache_matches_oracle(cache, bits, dt, keep, k, "bitmask")
    with pytest.raises(TypeError):
        dropit.dropit_produce(x.float(), 0.9, "relu")
    with pytest.raises(dropit.DropITError):
        dropit.dropit_compress_prepared(x, 0.9, prep[:64])
