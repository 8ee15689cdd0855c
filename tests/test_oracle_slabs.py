"""How much of a min-k mask is empty, counted on the oracle's selection (Sec. 3.2 keeps the recovered tensor dense
and runs the stock GEMM on it; a kernel that skipped empty regions of the mask would need empty regions).

The tensor has the value law of the ViT MLP's second Linear input (GELU of N(0,1)) with fewer tokens than the
benchmark's, which does not change the fractions.  Regions are token x channel blocks of the [M, Ca] input.
"""
import numpy as np
import pytest

import dropit_inputs as di
import oracle


def _empty_fraction(keep2d: np.ndarray, bt: int, bc: int) -> float:
    M, C = keep2d.shape
    blocks = keep2d[: M // bt * bt, : C // bc * bc].reshape(M // bt, bt, C // bc, bc)
    return float((~blocks.any(axis=(1, 3))).mean())


@pytest.mark.parametrize("gamma", [0.5, 0.8, 0.9, 0.95])
def test_no_slab_an_mma_could_skip_is_empty(gamma):
    case = di.small_linear(1024, 3072, 768, "bf16", gamma, "gelu")
    bits, dt = oracle.to_bits(di.make_x(case))
    keep, k = oracle.min_k(bits, gamma, dt)
    keep2d = keep.reshape(case.M, case.Ca).astype(bool)
    assert int(keep2d.sum()) == k
    # 16 tokens x 32 channels is the smallest piece of an operand tile that one K = 16 MMA step could leave out
    assert _empty_fraction(keep2d, 16, 32) == 0.0
    assert _empty_fraction(keep2d, 16, 128) == 0.0
    assert _empty_fraction(keep2d, 64, 256) == 0.0


def test_only_single_mask_words_are_sometimes_empty():
    case = di.small_linear(1024, 3072, 768, "bf16", 0.9, "gelu")
    bits, dt = oracle.to_bits(di.make_x(case))
    keep, _ = oracle.min_k(bits, 0.9, dt)
    words = _empty_fraction(keep.reshape(case.M, case.Ca).astype(bool), 1, 32)
    # (1 - 0.1)^32 = 3.4 % if the retained positions were independent; they very nearly are
    assert 0.025 < words < 0.045
