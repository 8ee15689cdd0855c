"""Pins for the oracle's min-k selection (Sec. 3.3 "Min-K Elements", Sec. 4.1 top-k of |a|)."""
import itertools
import os

import numpy as np
import pytest
import torch

import dropit_inputs as di
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def numpy_topk_keep(key, k):
    """Independent route: numpy's stable sort on descending key keeps equal keys in index order."""
    order = np.argsort(-(key.astype(np.int64)), kind="stable")
    keep = np.zeros(key.size, np.uint8)
    keep[order[:k]] = 1
    return keep


def test_exhaustive_tiny_tensors_rank_equals_sort_equals_numpy():
    alphabet = np.array([0x0000, 0x3F80, 0xBF80, 0x4000], np.uint16)  # +0, 1, -1, 2 as bf16
    for n in range(1, 7):
        for combo in itertools.product(range(4), repeat=n):
            x = alphabet[list(combo)]
            key = oracle.keys(x, oracle.BF16)
            for k in range(0, n + 1):
                a = oracle.select_rank(key, k)
                b = oracle.select_sort(key, k)
                c = numpy_topk_keep(key, k)
                assert (a == b).all() and (a == c).all(), (combo, k)


@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 257, 1000, 2048])
@pytest.mark.parametrize("levels", [2, 5, 1 << 15])
def test_random_with_ties_rank_equals_sort_equals_numpy(n, levels):
    rng = np.random.default_rng(n * 7 + levels)
    key = rng.integers(0, levels, n).astype(np.uint32)
    for k in sorted({0, 1, n // 10, n // 2, n - 1, n}):
        if k < 0:
            continue
        a = oracle.select_rank(key, k)
        b = oracle.select_sort(key, k)
        c = numpy_topk_keep(key, k)
        assert (a == b).all() and (a == c).all()
        assert int(a.sum()) == k


def check_invariants(key, keep, k):
    assert int(keep.sum()) == k
    if 0 < k < key.size:
        kept, dropped = key[keep == 1], key[keep == 0]
        t = kept.min()
        assert t >= dropped.max()
        # among elements equal to the threshold key, the retained ones are a prefix in flat-index order
        ties = keep[key == t]
        q = int(ties.sum())
        assert ties[:q].all() and not ties[q:].any()


@pytest.mark.parametrize("case", [di.small_linear(1500, 768, 8, "bf16", 0.9), di.small_linear(300, 3072, 8, "bf16", 0.9, "gelu"),
                                  di.small_conv(4, 64, 56, 56, 8, 1, 1, gamma=0.8), di.small_linear(256, 768, 8, "f32", 0.9)])
def test_invariants_on_workload_shaped_inputs(case):
    bits, dt = oracle.to_bits(di.make_x(case))
    keep, k = oracle.min_k(bits, case.gamma, dt)
    assert k == oracle.keep_count(bits.size, case.gamma)
    check_invariants(oracle.keys(bits, dt), keep, k)


def test_all_equal_tensor_keeps_the_lowest_indices():
    x = np.full(1000, 0x3F80, np.uint16)
    x[::2] |= 0x8000  # alternate the sign: magnitude is what counts
    keep, k = oracle.min_k(x, 0.7, oracle.BF16)
    assert k == 300
    assert keep[:300].all() and not keep[300:].any()


def test_strictly_increasing_magnitude_keeps_the_tail():
    x = torch.arange(1, 1001, dtype=torch.float32) * torch.where(torch.arange(1000) % 3 == 0, -1.0, 1.0)
    bits, dt = oracle.to_bits(x)
    keep, k = oracle.min_k(bits, 0.9, dt)
    assert k == 100 and keep[900:].all() and not keep[:900].any()
    keep, k = oracle.min_k(bits[::-1].copy(), 0.9, dt)
    assert keep[:100].all() and not keep[100:].any()


def test_sign_is_ignored_zero_inf_nan_order():
    f = np.array([0.0, -0.0, 1e-30, -3.0, np.inf, -np.inf, np.nan, 2.0], np.float32)
    key = oracle.keys(f.view(np.uint32), oracle.F32)
    assert key[0] == key[1] == 0
    assert key[4] == key[5] and key[6] > key[4] > key[3] > key[7] > key[2] > key[0]
    keep = oracle.select_sort(key, 3)
    assert list(np.flatnonzero(keep)) == [4, 5, 6]
    bf = np.array([0x0000, 0x8000, 0x7F80, 0xFF80, 0x7FC0, 0x0001], np.uint16)
    kb = oracle.keys(bf, oracle.BF16)
    assert kb[0] == kb[1] == 0 and kb[2] == kb[3] and kb[4] > kb[2] > kb[5] > kb[0]


def _golden_thresholds():
    out = {}
    with open(os.path.join(GOLDEN, "gaussian_thresholds.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            d, g, v = line.split()
            out[(d, float(g))] = float(v)
    return out


@pytest.mark.parametrize("dist,gamma", [("normal", 0.5), ("normal", 0.8), ("normal", 0.9), ("relu", 0.8), ("gelu", 0.9)])
def test_threshold_matches_the_closed_form_quantile(dist, gamma):
    gold = _golden_thresholds()[(dist, gamma)]
    case = di.small_linear(2048, 512, 8, "f32", gamma, dist)
    x = di.make_x(case)
    bits, dt = oracle.to_bits(x)
    keep, k = oracle.min_k(bits, gamma, dt)
    absx = x.abs().reshape(-1).numpy()
    t_lo, t_hi = absx[keep == 0].max(), absx[keep == 1].min()
    assert t_lo <= t_hi
    # quantile standard error ~ sqrt(p(1-p)/N)/pdf: about 2e-3 here
    assert abs(t_hi - gold) < 0.01, (t_hi, gold)
    # the same closed form from scipy rather than the stored text
    from scipy.stats import norm
    if dist == "normal":
        assert abs(norm.ppf(1 - (1 - gamma) / 2) - gold) < 1e-5


def test_retained_energy_of_a_gaussian_matches_closed_form():
    gold = _golden_thresholds()[("energy_normal", 0.9)]
    case = di.small_linear(2048, 512, 8, "f32", 0.9)
    x = di.make_x(case).reshape(-1).double().numpy()
    bits, dt = oracle.to_bits(di.make_x(case))
    keep, _ = oracle.min_k(bits, 0.9, dt)
    frac = (x[keep == 1] ** 2).sum() / (x ** 2).sum()
    assert abs(frac - gold) < 0.01


def test_a_planted_wrong_tie_break_is_caught():
    # a selection that breaks ties by HIGHER index satisfies count and order but must fail the prefix invariant
    key = np.array([5, 3, 3, 3, 1], np.uint32)
    bad = np.array([1, 0, 1, 1, 0], np.uint8)
    with pytest.raises(AssertionError):
        check_invariants(key, bad, 3)
    check_invariants(key, oracle.select_sort(key, 3), 3)
