"""Pins for the oracle's random dropping strategy (Sec. 3.3 "Random Elements") and its generator."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(v, 16) for v in r]
        assert oracle.philox4x32_10(w[0:4], w[4:6]).tolist() == w[6:10]


def test_philox_is_a_bijection_of_the_counter_on_a_slice():
    # for a fixed key the generator permutes the counter space: no two of 2^16 counters may collide
    key = [0x12345678, 0x9ABCDEF0]
    outs = {tuple(oracle.philox4x32_10([c, 7, 0, 0], key).tolist()) for c in range(1 << 16)}
    assert len(outs) == 1 << 16


def test_ranks_are_the_halves_of_the_blocks():
    n, seed = 1000, 0x0123456789ABCDEF
    ranks = oracle.random_ranks(n, seed)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for b in (0, 1, 17, 124):
        out = oracle.philox4x32_10([b, 0, 0, 0], key)
        halves = []
        for w in out.tolist():
            halves += [w & 0xFFFF, w >> 16]
        assert ranks[8 * b:8 * b + 8].tolist() == [h & 0x7FFF for h in halves]
    assert ranks.max() < (1 << 15)


def test_ranks_are_uniform():
    ranks = oracle.random_ranks(1 << 20, 1)
    counts = np.bincount(ranks >> 7, minlength=256).astype(np.float64)      # top 8 of the 15 bits
    expect = ranks.size / 256
    chi2 = ((counts - expect) ** 2 / expect).sum()
    assert chi2 < 350, chi2          # 255 degrees of freedom: mean 255, sd 22.6
    low = np.bincount(ranks & 0xFF, minlength=256).astype(np.float64)       # low 8 bits
    assert ((low - expect) ** 2 / expect).sum() < 350


@pytest.mark.parametrize("gamma", [0.0, 0.3, 0.9, 1.0])
def test_exact_count_and_order_rule(gamma):
    n, seed = 50_003, 42
    keep, k = oracle.random_k(n, gamma, seed)
    assert k == oracle.keep_count(n, gamma) == int(keep.sum())
    ranks = oracle.random_ranks(n, seed)
    if 0 < k < n:
        kept, dropped = ranks[keep == 1], ranks[keep == 0]
        t = kept.min()
        assert t >= dropped.max()                       # every retained rank >= every dropped rank
        ties = np.flatnonzero(ranks == t)
        kt = keep[ties]
        assert (np.diff(kt.astype(np.int8)) <= 0).all()  # among ties the retained ones are the lowest indices


def test_random_k_is_the_rank_definition_on_small_tensors():
    for n in (1, 7, 8, 9, 64, 333):
        for gamma in (0.1, 0.5, 0.9):
            keep, k = oracle.random_k(n, gamma, 3)
            assert (keep == oracle.select_rank(oracle.random_ranks(n, 3), k)).all()


def test_retained_positions_are_spread_evenly():
    n, gamma = 1 << 20, 0.9
    keep, k = oracle.random_k(n, gamma, 7)
    per = keep.reshape(64, -1).sum(axis=1).astype(np.float64)
    p = k / n
    var = (n / 64) * p * (1 - p)
    chi2 = ((per - k / 64) ** 2 / var).sum()
    assert chi2 < 110, chi2           # 63 degrees of freedom (the count is fixed): mean 63, sd 11.2


def test_seed_and_reproducibility():
    a, _ = oracle.random_k(10_000, 0.9, 1)
    b, _ = oracle.random_k(10_000, 0.9, 1)
    c, _ = oracle.random_k(10_000, 0.9, 2)
    assert (a == b).all() and (a != c).any()
    # independent of magnitude by construction; overlap of two seeds' retained sets is about k * (1 - gamma)
    overlap = int((a & c).sum())
    assert 50 < overlap < 160
