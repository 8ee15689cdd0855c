"""Pins for the oracle's cache encoders and recovery R(.) (Sec. 3.2 of arXiv 2202.13808)."""
import numpy as np
import pytest

import dropit_inputs as di
import oracle


@pytest.mark.parametrize("case", [di.small_linear(37, 129, 4, "bf16", 0.9), di.small_linear(64, 768, 4, "f32", 0.5),
                                  di.small_conv(2, 5, 7, 9, 3, 1, 1, gamma=0.8), di.small_linear(1, 1, 1, "bf16", 0.0)])
def test_bitmask_index_values_offsets_against_numpy(case):
    bits, dt = oracle.to_bits(di.make_x(case))
    keep, k = oracle.min_k(bits, case.gamma, dt)
    n = bits.size
    words = oracle.encode_bitmask(keep)
    pad = np.zeros(words.size * 32, np.uint8)
    pad[:n] = keep
    assert (np.packbits(pad, bitorder="little").view(np.uint32) == words).all()
    idx = oracle.encode_index32(keep)
    assert (idx == np.flatnonzero(keep).astype(np.int32)).all() and idx.size == k
    vals = oracle.pack_values(bits, keep, dt)
    assert (vals == bits[keep == 1]).all()
    for chunk in (128, 32, 1000):
        off = oracle.chunk_offsets(keep, chunk)
        cum = np.concatenate([[0], np.cumsum(keep, dtype=np.int64)])
        assert (off == cum[np.arange(off.size) * chunk]).all()
    # recovery leaves retained values untouched and fills the rest with +0
    rec_m = oracle.recover_from_bitmask(vals, words, n, dt)
    rec_i = oracle.recover_from_index32(vals, idx, n, dt)
    expect = np.where(keep == 1, bits, 0).astype(bits.dtype)
    assert (rec_m == expect).all() and (rec_i == expect).all()


def test_gamma_zero_roundtrip_is_identity_and_gamma_one_is_empty():
    case = di.small_linear(33, 65, 4, "bf16", 0.0)
    bits, dt = oracle.to_bits(di.make_x(case))
    keep, k = oracle.min_k(bits, 0.0, dt)
    assert k == bits.size and keep.all()
    assert (oracle.recover_from_bitmask(oracle.pack_values(bits, keep, dt), oracle.encode_bitmask(keep), bits.size, dt)
            == bits).all()
    keep, k = oracle.min_k(bits, 1.0, dt)
    assert k == 0 and not keep.any()
    assert oracle.pack_values(bits, keep, dt).size == 0
    assert not oracle.recover_from_bitmask(np.zeros(0, np.uint16), oracle.encode_bitmask(keep), bits.size, dt).any()


def test_negative_zero_and_nan_payloads_survive_packing():
    x = np.array([0x8000, 0x7FC1, 0xFFC2, 0x3F80, 0x0000, 0x8001], np.uint16)
    keep, k = oracle.min_k(x, 0.5, oracle.BF16)
    assert k == 3 and list(np.flatnonzero(keep)) == [1, 2, 3]
    assert list(oracle.pack_values(x, keep, oracle.BF16)) == [0x7FC1, 0xFFC2, 0x3F80]
