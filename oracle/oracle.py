"""numpy/ctypes binding of the C oracle (test infrastructure, see dropit_oracle.c).

Tensors cross this boundary as numpy arrays of RAW BITS: uint16 for bf16,
uint32 for fp32 (`to_bits` converts a torch CPU tensor).  Every function cites
the passage of arXiv 2202.13808 that it states.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

__all__ = [
    "BF16", "F32", "build", "to_bits", "keep_count", "keys", "select_rank", "select_sort", "min_k",
    "encode_bitmask", "encode_index32", "pack_values", "chunk_offsets", "recover_from_bitmask",
    "recover_from_index32", "fc_weight_grad", "fc_weight_grad_entries", "conv_weight_grad",
    "conv_weight_grad_entries", "num_threads", "bits_to_float64", "philox4x32_10", "random_ranks", "random_k",
    "ACT_IDENTITY", "ACT_RELU", "ACT_GELU", "round_to_bf16", "activation_table", "apply_table", "key_histogram_bf16",
    "q8_top_exponent", "q8_encode", "q8_decode",
]

BF16 = 0
F32 = 1
ACT_IDENTITY, ACT_RELU, ACT_GELU = 0, 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dropit_oracle.c")
_SO = os.path.join(_HERE, "libdropit_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile dropit_oracle.c with gcc into a shared object beside it."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-std=c99", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.oracle_keep_count.restype = ctypes.c_int64
            lib.oracle_keep_count.argtypes = [ctypes.c_int64, ctypes.c_double]
            lib.oracle_encode_index32.restype = ctypes.c_int64
            lib.oracle_pack_values.restype = ctypes.c_int64
            lib.oracle_select_sort.restype = ctypes.c_int
            lib.oracle_min_k.restype = ctypes.c_int
            lib.oracle_random_k.restype = ctypes.c_int
            lib.oracle_num_threads.restype = ctypes.c_int
            lib.oracle_q8_top_exponent.restype = ctypes.c_uint32
            lib.oracle_round_to_bf16.restype = ctypes.c_uint16
            lib.oracle_round_to_bf16.argtypes = [ctypes.c_double]
            _lib = lib
    return _lib


def _p(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return ctypes.c_void_p(a.ctypes.data)


def _i64(v):
    return ctypes.c_int64(int(v))


def _bits_dtype(dtype: int):
    return np.uint16 if dtype == BF16 else np.uint32


def _check_bits(x: np.ndarray, dtype: int) -> np.ndarray:
    x = np.ascontiguousarray(x)
    assert x.dtype == _bits_dtype(dtype), (x.dtype, dtype)
    return x


def to_bits(t):
    """torch CPU tensor (bf16 or fp32) -> (flat numpy array of raw bits, dtype code)."""
    import torch

    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).reshape(-1), BF16
    if t.dtype == torch.float32:
        return t.view(torch.int32).numpy().view(np.uint32).reshape(-1), F32
    raise TypeError(t.dtype)


def bits_to_float64(bits: np.ndarray, dtype: int) -> np.ndarray:
    """Exact widening of raw bits to float64 (bf16 is the top half of an fp32)."""
    if dtype == BF16:
        return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return bits.view(np.float32).astype(np.float64)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def keep_count(n: int, gamma: float) -> int:
    """Number of retained elements k = n - ceil(gamma*n - 1e-6) (Sec. 3.3, Sec. 4.1, Table 4)."""
    return int(_load().oracle_keep_count(int(n), float(gamma)))


def keys(x_bits: np.ndarray, dtype: int) -> np.ndarray:
    """Ordering key of |x| (Sec. 3.3): the bits with the sign cleared."""
    x_bits = _check_bits(x_bits, dtype)
    out = np.empty(x_bits.size, np.uint32)
    _load().oracle_keys(_p(x_bits), _i64(x_bits.size), ctypes.c_int(dtype), _p(out))
    return out


def select_rank(key_arr: np.ndarray, k: int) -> np.ndarray:
    """Literal rank definition of min-k (Sec. 3.3), O(n^2)."""
    key_arr = np.ascontiguousarray(key_arr, np.uint32)
    keep = np.empty(key_arr.size, np.uint8)
    _load().oracle_select_rank(_p(key_arr), _i64(key_arr.size), _i64(k), _p(keep))
    return keep


def select_sort(key_arr: np.ndarray, k: int) -> np.ndarray:
    """Same set through a sort on (key descending, flat index ascending) (Sec. 4.1: top-k of |a|)."""
    key_arr = np.ascontiguousarray(key_arr, np.uint32)
    keep = np.empty(key_arr.size, np.uint8)
    rc = _load().oracle_select_sort(_p(key_arr), _i64(key_arr.size), _i64(k), _p(keep))
    if rc != 0:
        raise MemoryError("oracle_select_sort")
    return keep


def min_k(x_bits: np.ndarray, gamma: float, dtype: int):
    """D(.) with the min-k strategy over the whole tensor -> (keep uint8[n], k)."""
    x_bits = _check_bits(x_bits, dtype)
    keep = np.empty(x_bits.size, np.uint8)
    k = ctypes.c_int64(0)
    rc = _load().oracle_min_k(_p(x_bits), _i64(x_bits.size), ctypes.c_double(gamma), ctypes.c_int(dtype), _p(keep),
                              ctypes.byref(k))
    if rc != 0:
        raise MemoryError("oracle_min_k")
    return keep, int(k.value)


def philox4x32_10(ctr, key) -> np.ndarray:
    """One block of Philox4x32-10 (Salmon et al., SC'11): 4 counter words, 2 key words -> 4 output words."""
    c = np.ascontiguousarray(ctr, np.uint32)
    k = np.ascontiguousarray(key, np.uint32)
    assert c.size == 4 and k.size == 2
    out = np.empty(4, np.uint32)
    _load().oracle_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def random_ranks(n: int, seed: int) -> np.ndarray:
    """15-bit rank of every element under `seed` (Sec. 3.3 "Random Elements")."""
    out = np.empty(int(n), np.uint32)
    _load().oracle_random_ranks(_i64(n), ctypes.c_uint64(int(seed) & (2 ** 64 - 1)), _p(out))
    return out


def random_k(n: int, gamma: float, seed: int):
    """D(.) with the random strategy (Sec. 3.3): the k highest ranks stay -> (keep uint8[n], k)."""
    keep = np.empty(int(n), np.uint8)
    k = ctypes.c_int64(0)
    rc = _load().oracle_random_k(_i64(n), ctypes.c_double(gamma), ctypes.c_uint64(int(seed) & (2 ** 64 - 1)), _p(keep),
                                 ctypes.byref(k))
    if rc != 0:
        raise MemoryError("oracle_random_k")
    return keep, int(k.value)


def encode_bitmask(keep: np.ndarray) -> np.ndarray:
    """X_r as an occupancy bitmask, bit (i mod 32) of word (i div 32) (Sec. 3.2)."""
    keep = np.ascontiguousarray(keep, np.uint8)
    words = np.empty((keep.size + 31) // 32, np.uint32)
    _load().oracle_encode_bitmask(_p(keep), _i64(keep.size), _p(words))
    return words


def encode_index32(keep: np.ndarray) -> np.ndarray:
    """X_r as ascending int32 flat indices (Sec. 4.1 coordinate format, App. A.7 int32)."""
    keep = np.ascontiguousarray(keep, np.uint8)
    idx = np.empty(int(keep.sum()), np.int32)
    c = _load().oracle_encode_index32(_p(keep), _i64(keep.size), _p(idx))
    assert c == idx.size
    return idx


def pack_values(x_bits: np.ndarray, keep: np.ndarray, dtype: int) -> np.ndarray:
    """a_Xr: retained values, raw bits, ascending flat index (Sec. 3.2)."""
    x_bits = _check_bits(x_bits, dtype)
    keep = np.ascontiguousarray(keep, np.uint8)
    vals = np.empty(int(keep.sum()), _bits_dtype(dtype))
    c = _load().oracle_pack_values(_p(x_bits), _p(keep), _i64(x_bits.size), ctypes.c_int(dtype), _p(vals))
    assert c == vals.size
    return vals


def chunk_offsets(keep: np.ndarray, chunk: int) -> np.ndarray:
    """offsets[c] = retained elements with flat index < c*chunk."""
    keep = np.ascontiguousarray(keep, np.uint8)
    out = np.empty((keep.size + chunk - 1) // chunk, np.uint32)
    _load().oracle_chunk_offsets(_p(keep), _i64(keep.size), _i64(chunk), _p(out))
    return out


def recover_from_bitmask(values: np.ndarray, words: np.ndarray, n: int, dtype: int) -> np.ndarray:
    """R(a-hat): dense tensor with dropped positions = +0 (Sec. 3.2)."""
    values = _check_bits(values, dtype)
    words = np.ascontiguousarray(words, np.uint32)
    out = np.empty(n, _bits_dtype(dtype))
    _load().oracle_recover_from_bitmask(_p(values), _p(words), _i64(n), ctypes.c_int(dtype), _p(out))
    return out


def recover_from_index32(values: np.ndarray, idx: np.ndarray, n: int, dtype: int) -> np.ndarray:
    values = _check_bits(values, dtype)
    idx = np.ascontiguousarray(idx, np.int32)
    out = np.empty(n, _bits_dtype(dtype))
    _load().oracle_recover_from_index32(_p(values), _p(idx), _i64(idx.size), _i64(n), ctypes.c_int(dtype), _p(out))
    return out


def fc_weight_grad(dy_bits, x_bits, keep, M, Ca, Cz, dtype) -> np.ndarray:
    """Eq. 6: dW[j,c] = sum over retained (n,c) of dY[n,j] a[n,c]; float64 [Cz, Ca]."""
    dy_bits = _check_bits(dy_bits, dtype)
    x_bits = _check_bits(x_bits, dtype)
    keep = np.ascontiguousarray(keep, np.uint8)
    assert dy_bits.size == M * Cz and x_bits.size == M * Ca and keep.size == M * Ca
    dw = np.empty((Cz, Ca), np.float64)
    _load().oracle_fc_weight_grad(_p(dy_bits), _p(x_bits), _p(keep), _i64(M), _i64(Ca), _i64(Cz), ctypes.c_int(dtype),
                                  _p(dw))
    return dw


def fc_weight_grad_entries(dy_bits, x_bits, keep, M, Ca, Cz, dtype, js, cs) -> np.ndarray:
    """Eq. 6 for the listed output entries only."""
    dy_bits = _check_bits(dy_bits, dtype)
    x_bits = _check_bits(x_bits, dtype)
    keep = np.ascontiguousarray(keep, np.uint8)
    js = np.ascontiguousarray(js, np.int64)
    cs = np.ascontiguousarray(cs, np.int64)
    out = np.empty(js.size, np.float64)
    _load().oracle_fc_weight_grad_entries(_p(dy_bits), _p(x_bits), _p(keep), _i64(M), _i64(Ca), _i64(Cz),
                                          ctypes.c_int(dtype), _p(js), _p(cs), _i64(js.size), _p(out))
    return out


def conv_weight_grad(dy_bits, x_bits, keep, B, Ca, H, W, Cz, R, S, stride, pad, dtype) -> np.ndarray:
    """Eq. 4-5 retained term, element-wise mask on the input; float64 [Cz, Ca, R, S]."""
    dy_bits = _check_bits(dy_bits, dtype)
    x_bits = _check_bits(x_bits, dtype)
    keep = np.ascontiguousarray(keep, np.uint8)
    Ho = (H + 2 * pad - R) // stride + 1
    Wo = (W + 2 * pad - S) // stride + 1
    assert x_bits.size == B * Ca * H * W and dy_bits.size == B * Cz * Ho * Wo
    dw = np.empty((Cz, Ca, R, S), np.float64)
    _load().oracle_conv_weight_grad(_p(dy_bits), _p(x_bits), _p(keep), _i64(B), _i64(Ca), _i64(H), _i64(W), _i64(Cz),
                                    _i64(R), _i64(S), _i64(stride), _i64(pad), ctypes.c_int(dtype), _p(dw))
    return dw


def conv_weight_grad_entries(dy_bits, x_bits, keep, B, Ca, H, W, Cz, R, S, stride, pad, dtype, js, cs, us,
                             vs) -> np.ndarray:
    dy_bits = _check_bits(dy_bits, dtype)
    x_bits = _check_bits(x_bits, dtype)
    keep = np.ascontiguousarray(keep, np.uint8)
    js, cs, us, vs = (np.ascontiguousarray(a, np.int64) for a in (js, cs, us, vs))
    out = np.empty(js.size, np.float64)
    _load().oracle_conv_weight_grad_entries(_p(dy_bits), _p(x_bits), _p(keep), _i64(B), _i64(Ca), _i64(H), _i64(W),
                                            _i64(Cz), _i64(R), _i64(S), _i64(stride), _i64(pad), ctypes.c_int(dtype),
                                            _p(js), _p(cs), _p(us), _p(vs), _i64(js.size), _p(out))
    return out


def round_to_bf16(v: float) -> int:
    """A double rounded once to bf16, ties to even; the result's bits."""
    return int(_load().oracle_round_to_bf16(float(v)))


def activation_table(act: int) -> np.ndarray:
    """The element-wise producer in front of a conv / fc input (Sec. 3.5) as a table over all bf16 bit
    patterns: table[b] = bits of act(value of b), act in double, rounded once."""
    table = np.empty(65536, np.uint16)
    _load().oracle_activation_table(ctypes.c_int(int(act)), _p(table))
    return table


def apply_table(table: np.ndarray, x_bits: np.ndarray) -> np.ndarray:
    """y[i] = table[x[i]] on raw bf16 bits."""
    table = _check_bits(table, BF16)
    x = _check_bits(x_bits, BF16)
    assert table.size == 65536
    y = np.empty_like(x)
    _load().oracle_apply_table(_p(table), _p(x), _i64(x.size), _p(y))
    return y


def key_histogram_bf16(x_bits: np.ndarray) -> np.ndarray:
    """hist[key] = number of elements whose bits with the sign cleared equal key (32768 bins)."""
    x = _check_bits(x_bits, BF16)
    hist = np.zeros(32768, np.uint64)
    _load().oracle_key_histogram_bf16(_p(x), _i64(x.size), _p(hist))
    return hist


def q8_top_exponent(values_bits: np.ndarray) -> int:
    """Largest exponent field among the finite values: the scale of the tensor's 8-bit codes."""
    v = _check_bits(values_bits, BF16)
    return int(_load().oracle_q8_top_exponent(_p(v), _i64(v.size)))


def q8_encode(values_bits: np.ndarray, e_top: int) -> np.ndarray:
    """Retained bf16 values as 8-bit codes sign | e3 | m4 under the shared top exponent (Sec. 1, Table 5: DropIT
    combined with 8-bit quantisation, here on DropIT's own payload)."""
    v = _check_bits(values_bits, BF16)
    out = np.empty(v.size, np.uint8)
    _load().oracle_q8_encode(_p(v), _i64(v.size), ctypes.c_uint32(int(e_top)), _p(out))
    return out


def q8_decode(codes: np.ndarray, e_top: int) -> np.ndarray:
    """The bf16 values that the 8-bit codes stand for."""
    c = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty(c.size, np.uint16)
    _load().oracle_q8_decode(_p(c), _i64(c.size), ctypes.c_uint32(int(e_top)), _p(out))
    return out
