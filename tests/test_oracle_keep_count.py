"""Pins for the oracle's keep-count rule (Sec. 3.3, Sec. 4.1, Table 4 of arXiv 2202.13808)."""
import os
from fractions import Fraction

import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

# (N, gamma as an exact decimal string)
CASES = [
    (256 * 768, "0.9"), (12608 * 768, "0.9"), (12608 * 3072, "0.9"),
    (64 * 256 * 56 * 56, "0.8"), (64 * 64 * 56 * 56, "0.8"),
    (32768 * 768, "0.5"), (32768 * 768, "0.8"), (32768 * 768, "0.9"),
    (32768 * 3072, "0.5"), (32768 * 3072, "0.8"), (32768 * 3072, "0.9"),
    (10, "0.9"), (10, "0.1"), (7, "0.5"), (1, "0.5"), (1, "0.0"), (1, "1.0"), (3, "0.3333"), (1000, "0.7"),
    (999, "0.999"), (12345, "0.6"), (2 ** 31 - 1, "0.9"),
]


@pytest.mark.parametrize("n,gs", CASES)
def test_keep_count_is_exact_floor_of_budget(n, gs):
    # never keep more than the (1-gamma) budget: k = floor((1-gamma) N) in exact rational arithmetic
    g = Fraction(gs)
    expect = (n * (1 - g)).__floor__()
    assert oracle.keep_count(n, float(gs)) == expect


def test_keep_count_values_at_the_evaluation_shapes():
    # worked by hand: 0.1 * 196608 = 19660.8 ; 0.1 * 9682944 = 968294.4 ; 0.2 * 51380224 = 10276044.8
    assert oracle.keep_count(196608, 0.9) == 19660
    assert oracle.keep_count(9682944, 0.9) == 968294
    assert oracle.keep_count(38731776, 0.9) == 3873177
    assert oracle.keep_count(51380224, 0.8) == 10276044
    assert oracle.keep_count(12845056, 0.8) == 2569011
    assert oracle.keep_count(25165824, 0.5) == 12582912


def test_gamma_zero_keeps_all_and_one_keeps_none():
    # Table 2 column "0% (Baseline)": nothing dropped
    for n in (1, 2, 31, 32, 33, 1000, 12608 * 768):
        assert oracle.keep_count(n, 0.0) == n
        assert oracle.keep_count(n, 1.0) == 0


def test_keep_count_monotone_in_gamma():
    n = 1237
    prev = n
    for i in range(0, 1001):
        k = oracle.keep_count(n, i / 1000.0)
        assert 0 <= k <= prev
        prev = k


def test_table4_memory_falls_precisely_by_gamma():
    rows = []
    with open(os.path.join(GOLDEN, "table4_cached_fc_tensors.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            gp, gb = line.split()
            rows.append((int(gp), float(gb)))
    dense = dict(rows)[0]
    n = 1024 * 197 * 384  # one DeiT-S FC input at batch 1024
    for gp, gb in rows:
        k = oracle.keep_count(n, gp / 100.0)
        assert round(dense * k / n, 2) == pytest.approx(gb, abs=0.0051)


def test_int32_index_breaks_even_at_half():
    # App. A.7: an int32 index costs as much as an fp32 value, so the coordinate format only pays for gamma > 0.5
    n = 4096
    for gp in range(0, 101, 5):
        k = oracle.keep_count(n, gp / 100.0)
        coo_bytes = k * 4 + k * 4
        assert (coo_bytes < n * 4) == (gp > 50)
