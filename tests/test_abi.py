"""The C-ABI library loads, exports what include/dropit.h declares, and its host-only calls agree with the oracle."""
import ctypes
import os
import re

import pytest

import oracle
from paper_2202_13808_b200 import _lib, build as build_mod
import paper_2202_13808_b200 as dropit

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return _lib.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dropit.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dropit_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"dropit_compress", "dropit_weight_grad", "dropit_conv_weight_grad", "dropit_decompress"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(_lib.SIGNATURES), set(names) ^ set(_lib.SIGNATURES)


def test_version_and_status_strings(lib):
    assert dropit.dropit_version() >= 100
    assert dropit.dropit_status_string(0) == "DROPIT_OK"
    assert dropit.dropit_status_string(5) == "DROPIT_ERR_TIMEOUT"


@pytest.mark.parametrize("n", [0, 1, 7, 10, 1000, 196608, 9682944, 38731776, 51380224, 2 ** 31 - 1])
@pytest.mark.parametrize("gamma", [0.0, 0.1, 0.5, 0.8, 0.9, 0.999, 1.0])
def test_keep_count_matches_the_oracle_rule(lib, n, gamma):
    assert dropit.dropit_keep_count(n, gamma) == oracle.keep_count(n, gamma)


def test_keep_count_rejects_bad_arguments(lib):
    assert dropit.dropit_keep_count(-1, 0.5) == -1
    assert dropit.dropit_keep_count(10, -0.1) == -1
    assert dropit.dropit_keep_count(10, 1.5) == -1
    assert dropit.dropit_keep_count(10, float("nan")) == -1


def test_cache_sizes(lib):
    n = 12608 * 768
    v, m, o, w = dropit.dropit_cache_sizes(n, 0.9, dropit.BF16, dropit.FMT_BITMASK)
    k = oracle.keep_count(n, 0.9)
    assert v == 2 * k and m == 4 * ((n + 31) // 32) and o == 4 * ((n + 127) // 128) and w > 0
    v, m, o, w = dropit.dropit_cache_sizes(n, 0.9, dropit.F32, dropit.FMT_INDEX32)
    assert v == 4 * k and m == 4 * k
    # bitmask cache at gamma = 0.9 is 16.25% of dense bf16 (+ the seek table)
    v, m, o, w = dropit.dropit_cache_sizes(n, 0.9, dropit.BF16, dropit.FMT_BITMASK)
    assert abs((v + m) / (2 * n) - 0.1625) < 1e-4
    with pytest.raises(dropit.DropITError):
        dropit.dropit_cache_sizes(-1, 0.9, 0, 0)
    with pytest.raises(dropit.DropITError):
        dropit.dropit_cache_sizes(2 ** 31, 0.9, 0, 0)
    with pytest.raises(dropit.DropITError):
        dropit.dropit_cache_sizes(10, 2.0, 0, 0)
    with pytest.raises(dropit.DropITError):
        dropit.dropit_cache_sizes(10, 0.5, 7, 0)


def test_host_side_argument_validation_needs_no_gpu(lib):
    null = ctypes.c_void_p(0)
    # null input
    assert lib.dropit_compress(null, 100, 0.5, 0, 0, null, null, null, null, 0, null, null) == 1
    # gamma out of range / NaN
    assert lib.dropit_compress(null, 100, 1.5, 0, 0, null, null, null, null, 0, null, null) == 1
    assert lib.dropit_compress(null, 100, float("nan"), 0, 0, null, null, null, null, 0, null, null) == 1
    # empty tensor is a no-op
    assert lib.dropit_compress(null, 0, 0.5, 0, 0, null, null, null, null, 0, null, null) == 0
    # misaligned pointer
    assert lib.dropit_compress(ctypes.c_void_p(8), 100, 0.5, 0, 0, ctypes.c_void_p(16), ctypes.c_void_p(16),
                               ctypes.c_void_p(16), ctypes.c_void_p(16), 1 << 20, null, null) == 1
    # workspace too small
    assert lib.dropit_compress(ctypes.c_void_p(16), 100, 0.5, 0, 0, ctypes.c_void_p(16), ctypes.c_void_p(16),
                               ctypes.c_void_p(16), ctypes.c_void_p(16), 8, null, null) == 3
    # dilation other than 1
    assert lib.dropit_conv_weight_grad(null, null, null, null, 1, 1, 4, 4, 1, 3, 3, 1, 1, 2, 1, 0, 0,
                                       ctypes.c_void_p(16), 0, null, 0, null, null) == 2
    # bad shapes
    assert lib.dropit_weight_grad(null, null, null, null, 4, 0, 4, 1, 0, 0, ctypes.c_void_p(16), 0, null, 0, null,
                                  null) == 1
    out = ctypes.c_size_t(0)
    assert lib.dropit_conv_weight_grad_workspace(1, 1, 2, 2, 1, 5, 5, 1, 0, 0, 0, ctypes.byref(out)) == 1


def test_binding_refuses_cpu_tensors(lib):
    import torch
    with pytest.raises(ValueError):
        dropit.dropit_compress(torch.zeros(8), 0.5)
