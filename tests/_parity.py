"""Helpers shared by the GPU parity tests: run the oracle on the same seeded input and compare."""
import numpy as np
import torch

import dropit_inputs as di
import oracle
import paper_2202_13808_b200 as dropit


def np_bits(t: torch.Tensor) -> np.ndarray:
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).reshape(-1)
    if t.dtype == torch.float32:
        return t.view(torch.int32).numpy().view(np.uint32).reshape(-1)
    if t.dtype == torch.int32:
        return t.numpy().view(np.uint32).reshape(-1)
    raise TypeError(t.dtype)


def oracle_cache(x_cpu: torch.Tensor, gamma: float):
    bits, dt = oracle.to_bits(x_cpu)
    keep, k = oracle.min_k(bits, gamma, dt)
    return bits, dt, keep, k


def assert_cache_matches_oracle(cache, bits, dt, keep, k, fmt):
    """Bit-exact: retained set (mask or indices), packed values, chunk offsets."""
    assert cache.k == k == dropit.dropit_keep_count(bits.size, cache.gamma)
    assert cache.values.numel() == k
    got_vals = np_bits(cache.values)
    exp_vals = oracle.pack_values(bits, keep, dt)
    if fmt == "bitmask":
        got = np_bits(cache.meta)
        exp = oracle.encode_bitmask(keep)
        assert got.size == exp.size
        bad = np.flatnonzero(got != exp)
        assert bad.size == 0, "mask differs at %d words, first %s" % (bad.size, bad[:5])
    else:
        got = cache.meta.cpu().numpy()
        exp = oracle.encode_index32(keep)
        assert got.size == exp.size == k
        bad = np.flatnonzero(got != exp)
        assert bad.size == 0, "indices differ at %d, first %s" % (bad.size, bad[:5])
    badv = np.flatnonzero(got_vals != exp_vals)
    assert badv.size == 0, "values differ at %d, first %s" % (badv.size, badv[:5])
    got_off = np_bits(cache.offsets)
    exp_off = oracle.chunk_offsets(keep, dropit.CHUNK)
    assert got_off.size == exp_off.size
    assert (got_off == exp_off).all(), "offsets differ"


def max_rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max |got - ref| / max |ref| (max-norm relative error)."""
    denom = np.abs(ref).max()
    if denom == 0:
        return float(np.abs(got).max())
    return float(np.abs(got.astype(np.float64) - ref).max() / denom)
