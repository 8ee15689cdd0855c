"""Torch-facing binding of the C ABI in include/dropit.h.

Argument marshalling only: every step (selection, packing, recovery, weight gradients) runs in
the CUDA library.  torch supplies device memory and the current stream.
"""
from __future__ import annotations

import contextlib
import ctypes
import functools
import os
from dataclasses import dataclass
from typing import Optional, Tuple

import torch

from . import _lib

BF16, F32 = 0, 1
FMT_BITMASK, FMT_INDEX32 = 0, 1
CHUNK = 128

_DTYPE_CODE = {torch.bfloat16: BF16, torch.float32: F32}
_FMT_CODE = {"bitmask": FMT_BITMASK, "index32": FMT_INDEX32, FMT_BITMASK: FMT_BITMASK, FMT_INDEX32: FMT_INDEX32}


class DropITError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s" % (where, dropit_status_string(code)))


def library_path() -> str:
    return _lib.LIB_PATH


def dropit_version() -> int:
    return int(_lib.load().dropit_version())


def dropit_launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(_lib.load().dropit_launch_count())


def dropit_status_string(code: int) -> str:
    return _lib.load().dropit_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != 0:
        raise DropITError(code, where)


@functools.lru_cache(maxsize=4096)
def dropit_keep_count(n: int, gamma: float) -> int:
    """k = n - ceil(gamma*n - 1e-6): retained elements at drop ratio gamma (Sec. 3.3, Sec. 4.1)."""
    return int(_lib.load().dropit_keep_count(int(n), float(gamma)))


@functools.lru_cache(maxsize=4096)
def dropit_cache_sizes(n: int, gamma: float, dtype: int, fmt: int) -> Tuple[int, int, int, int]:
    """(values_bytes, meta_bytes, offsets_bytes, workspace_bytes) for dropit_compress."""
    out = [ctypes.c_size_t(0) for _ in range(4)]
    _check(_lib.load().dropit_cache_sizes(int(n), float(gamma), int(dtype), int(fmt), *[ctypes.byref(o) for o in out]),
           "dropit_cache_sizes")
    return tuple(int(o.value) for o in out)


@dataclass
class DropITCache:
    """a-hat = {a_Xr, X_r} (Sec. 3.2): packed retained values + occupancy mask or int32 indices."""
    values: torch.Tensor        # k elements, input dtype
    meta: torch.Tensor          # int32 words: bitmask (ceil(n/32)) or ascending flat indices (k)
    offsets: torch.Tensor       # int32: retained count before each 128-element chunk
    n: int
    k: int
    shape: Tuple[int, ...]
    dtype: torch.dtype
    fmt: int
    gamma: float

    codes: Optional[torch.Tensor] = None    # 8-bit codes of the values (dropit_quantize_cache); then `values` is None
    scale: Optional[torch.Tensor] = None    # the codes' shared top exponent (one int32 on the device)

    @property
    def nbytes(self) -> int:
        parts = (self.values, self.meta, self.offsets, self.codes, self.scale)
        return sum(t.numel() * t.element_size() for t in parts if t is not None)


_status_words = {}


def _status_word(device: torch.device) -> torch.Tensor:
    key = (device.type, device.index)
    if key not in _status_words:
        _status_words[key] = torch.zeros(4, dtype=torch.int32, device=device)
    return _status_words[key]


def check_device_status(device=None) -> None:
    """Synchronise and raise if a kernel reported a bounded wait running out."""
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    w = _status_word(device)
    code = int(w[0].item())
    if code != 0:
        w.zero_()
        raise DropITError(code, "device status")


def _ptr(t: Optional[torch.Tensor]):
    return ctypes.c_void_p(0 if t is None or t.numel() == 0 else t.data_ptr())


def _stream_ptr(device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def _on_device(dev: torch.device):
    """Make `dev` the current CUDA device for the call; free when it already is."""
    if dev.index is None or dev.index == torch.cuda.current_device():
        return contextlib.nullcontext()
    return torch.cuda.device(dev)


def _require_cuda(t: torch.Tensor, name: str):
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor (there is no CPU path)" % name)
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    if t.dtype not in _DTYPE_CODE:
        raise TypeError("%s: dtype %s is not supported (bf16 or fp32)" % (name, t.dtype))


def dropit_compress(x: torch.Tensor, gamma: float, fmt="bitmask", workspace: Optional[torch.Tensor] = None) -> DropITCache:
    """D(a), min-k (Sec. 3.3): retain the k largest-|x| elements of the whole tensor."""
    _require_cuda(x, "x")
    lib = _lib.load()
    fmt = _FMT_CODE[fmt]
    dt = _DTYPE_CODE[x.dtype]
    n = x.numel()
    vb, mb, ob, wb = dropit_cache_sizes(n, gamma, dt, fmt)
    k = dropit_keep_count(n, gamma)
    dev = x.device
    values = torch.empty(vb // x.element_size(), dtype=x.dtype, device=dev)
    meta = torch.empty(mb // 4, dtype=torch.int32, device=dev)
    offsets = torch.empty(ob // 4, dtype=torch.int32, device=dev)
    if workspace is None or workspace.numel() < wb:
        workspace = torch.empty(max(wb, 16), dtype=torch.uint8, device=dev)
    with _on_device(dev):
        code = lib.dropit_compress(_ptr(x), n, float(gamma), dt, fmt, _ptr(values), _ptr(meta), _ptr(offsets),
                                   _ptr(workspace), workspace.numel(), _ptr(_status_word(dev)), _stream_ptr(dev))
    _check(code, "dropit_compress")
    return DropITCache(values, meta, offsets, n, k, tuple(x.shape), x.dtype, fmt, float(gamma))


def dropit_quantize_cache(cache: DropITCache) -> DropITCache:
    """The same cache with its bf16 values replaced by 8-bit codes (sign, 3 exponent bits, 4 mantissa bits under the
    tensor's top exponent): 1 byte per retained element.  Mask / indices and seek table are shared with `cache`."""
    if cache.dtype != torch.bfloat16:
        raise TypeError("8-bit codes are defined for bf16 caches")
    if cache.values is None:
        return cache
    dev = cache.values.device if cache.k else cache.offsets.device
    codes = torch.empty(cache.k, dtype=torch.uint8, device=dev)
    scale = torch.zeros(1, dtype=torch.int32, device=dev)
    with _on_device(dev):
        code = _lib.load().dropit_quantize_values(_ptr(cache.values), cache.k, _ptr(codes), _ptr(scale), _stream_ptr(dev))
    _check(code, "dropit_quantize_values")
    return DropITCache(None, cache.meta, cache.offsets, cache.n, cache.k, cache.shape, cache.dtype, cache.fmt,
                       cache.gamma, codes, scale)


def dropit_dequantize_cache(cache: DropITCache) -> DropITCache:
    """A cache with bf16 values again (exactly the values the codes stand for); a no-op for an unquantised cache."""
    if cache.values is not None:
        return cache
    dev = cache.scale.device
    values = torch.empty(cache.k, dtype=torch.bfloat16, device=dev)
    with _on_device(dev):
        code = _lib.load().dropit_dequantize_values(_ptr(cache.codes), _ptr(cache.scale), cache.k, _ptr(values),
                                                    _stream_ptr(dev))
    _check(code, "dropit_dequantize_values")
    return DropITCache(values, cache.meta, cache.offsets, cache.n, cache.k, cache.shape, cache.dtype, cache.fmt, cache.gamma)


ACT_IDENTITY, ACT_RELU, ACT_TABLE = 0, 1, 2
TABLE_IDENTITY, TABLE_RELU, TABLE_GELU = 0, 1, 2
_TABLE_KIND = {"identity": TABLE_IDENTITY, "relu": TABLE_RELU, "gelu": TABLE_GELU}
_tables = {}


def dropit_activation_table(kind: str, device) -> torch.Tensor:
    """bf16 -> bf16 table of an element-wise activation over all 65536 bit patterns (int16 tensor on `device`),
    every entry evaluated in double and rounded once; built on the device the first time it is asked for."""
    device = torch.device(device)
    key = (kind, device.type, _device_index(device))
    if key not in _tables:
        t = torch.empty(65536, dtype=torch.int16, device=device)
        with _on_device(device):
            code = _lib.load().dropit_activation_table(_TABLE_KIND[kind], _ptr(t), _stream_ptr(device))
        _check(code, "dropit_activation_table")
        _tables[key] = t
    return _tables[key]


@functools.lru_cache(maxsize=4096)
def dropit_produce_workspace(n: int) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib.load().dropit_produce_workspace(int(n), ctypes.byref(out)), "dropit_produce_workspace")
    return int(out.value)


def dropit_produce(x: torch.Tensor, gamma: float, act: str = "identity", table: Optional[torch.Tensor] = None,
                   want_y: bool = True):
    """The element-wise layer in front of a conv / fc input (Sec. 3.5) fused with the first half of the selection:
    returns (y, prep) with y = act(x) (None when act is "identity" and want_y is False) and prep the selection
    statistics of y for drop ratio gamma, to be handed to dropit_compress_prepared.
    act: "identity", "relu", "gelu", or "table" with an int16 tensor of 65536 bf16 patterns."""
    _require_cuda(x, "x")
    if x.dtype != torch.bfloat16:
        raise TypeError("dropit_produce takes bf16 tensors")
    dev = x.device
    if act == "gelu":
        table, code_act = dropit_activation_table("gelu", dev), ACT_TABLE
    elif act == "table":
        if table is None or table.numel() != 65536 or table.dtype != torch.int16 or table.device != dev:
            raise ValueError("table must be an int16 tensor of 65536 bf16 patterns on the input's device")
        code_act = ACT_TABLE
    else:
        code_act = {"identity": ACT_IDENTITY, "relu": ACT_RELU}[act]
    n = x.numel()
    y = torch.empty_like(x) if (want_y or code_act != ACT_IDENTITY) else None
    prep = torch.empty(max(dropit_produce_workspace(n), 16), dtype=torch.uint8, device=dev)
    with _on_device(dev):
        code = _lib.load().dropit_produce(_ptr(x), n, float(gamma), code_act, _ptr(table), _ptr(y), _ptr(prep),
                                          prep.numel(), _stream_ptr(dev))
    _check(code, "dropit_produce")
    return y, prep


def dropit_compress_prepared(y: torch.Tensor, gamma: float, prep: torch.Tensor, fmt="bitmask",
                             workspace: Optional[torch.Tensor] = None) -> DropITCache:
    """dropit_compress of a tensor whose selection statistics dropit_produce has already taken: one read of y."""
    _require_cuda(y, "y")
    if y.dtype != torch.bfloat16:
        raise TypeError("dropit_compress_prepared takes bf16 tensors")
    lib = _lib.load()
    fmt = _FMT_CODE[fmt]
    n = y.numel()
    vb, mb, ob, wb = dropit_cache_sizes(n, gamma, BF16, fmt)
    k = dropit_keep_count(n, gamma)
    dev = y.device
    values = torch.empty(vb // 2, dtype=torch.bfloat16, device=dev)
    meta = torch.empty(mb // 4, dtype=torch.int32, device=dev)
    offsets = torch.empty(ob // 4, dtype=torch.int32, device=dev)
    if workspace is None or workspace.numel() < wb:
        workspace = torch.empty(max(wb, 16), dtype=torch.uint8, device=dev)
    with _on_device(dev):
        code = lib.dropit_compress_prepared(_ptr(y), n, float(gamma), fmt, _ptr(values), _ptr(meta), _ptr(offsets),
                                            _ptr(prep), prep.numel(), _ptr(workspace), workspace.numel(),
                                            _ptr(_status_word(dev)), _stream_ptr(dev))
    _check(code, "dropit_compress_prepared")
    return DropITCache(values, meta, offsets, n, k, tuple(y.shape), y.dtype, fmt, float(gamma))


@functools.lru_cache(maxsize=4096)
def dropit_compress_random_workspace(n: int, gamma: float) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib.load().dropit_compress_random_workspace(int(n), float(gamma), ctypes.byref(out)),
           "dropit_compress_random_workspace")
    return int(out.value)


def dropit_compress_random(x: torch.Tensor, gamma: float, seed: int, fmt="bitmask",
                           workspace: Optional[torch.Tensor] = None) -> DropITCache:
    """D(a), random strategy (Sec. 3.3 "Random Elements"): k elements chosen by Philox rank under `seed`."""
    _require_cuda(x, "x")
    lib = _lib.load()
    fmt = _FMT_CODE[fmt]
    dt = _DTYPE_CODE[x.dtype]
    n = x.numel()
    vb, mb, ob, _ = dropit_cache_sizes(n, gamma, dt, fmt)
    wb = dropit_compress_random_workspace(n, gamma)
    k = dropit_keep_count(n, gamma)
    dev = x.device
    values = torch.empty(vb // x.element_size(), dtype=x.dtype, device=dev)
    meta = torch.empty(mb // 4, dtype=torch.int32, device=dev)
    offsets = torch.empty(ob // 4, dtype=torch.int32, device=dev)
    if workspace is None or workspace.numel() < wb:
        workspace = torch.empty(max(wb, 16), dtype=torch.uint8, device=dev)
    with _on_device(dev):
        code = lib.dropit_compress_random(_ptr(x), n, float(gamma), int(seed) & (2 ** 64 - 1), dt, fmt, _ptr(values),
                                          _ptr(meta), _ptr(offsets), _ptr(workspace), workspace.numel(),
                                          _ptr(_status_word(dev)), _stream_ptr(dev))
    _check(code, "dropit_compress_random")
    return DropITCache(values, meta, offsets, n, k, tuple(x.shape), x.dtype, fmt, float(gamma))


def dropit_decompress(cache: DropITCache, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """R(a-hat) (Sec. 3.2): dense tensor, dropped positions +0; written into `out` when given."""
    cache = dropit_dequantize_cache(cache)
    lib = _lib.load()
    dev = cache.offsets.device if cache.offsets.numel() else cache.values.device
    if out is None:
        out = torch.empty(cache.shape, dtype=cache.dtype, device=dev)
    elif out.numel() != cache.n or out.dtype != cache.dtype or not out.is_contiguous() or out.device != dev:
        raise ValueError("out must be a contiguous %s tensor of %d elements on %s" % (cache.dtype, cache.n, dev))
    with _on_device(dev):
        code = lib.dropit_decompress(_ptr(cache.values), _ptr(cache.meta), _ptr(cache.offsets), cache.n, cache.k,
                                     _DTYPE_CODE[cache.dtype], cache.fmt, _ptr(out), _stream_ptr(dev))
    _check(code, "dropit_decompress")
    return out


def _device_index(device) -> int:
    if device is None:
        return torch.cuda.current_device()
    device = torch.device(device)
    return torch.cuda.current_device() if device.index is None else device.index


@functools.lru_cache(maxsize=4096)
def _weight_grad_workspace(M: int, Ca: int, Cz: int, dtype: int, fmt: int, dev_index: int, path: str) -> int:
    out = ctypes.c_size_t(0)
    with _on_device(torch.device("cuda", dev_index)):
        code = _lib.load().dropit_weight_grad_workspace(M, Ca, Cz, dtype, fmt, ctypes.byref(out))
    _check(code, "dropit_weight_grad_workspace")
    return int(out.value)


def dropit_weight_grad_workspace(M: int, Ca: int, Cz: int, dtype: int, fmt: int, device=None) -> int:
    """Scratch bytes of dropit_weight_grad on `device` (the plan depends on the device's SM count, and on the
    kernel that DROPIT_WG_PATH asks for, which the library reads at every call)."""
    return _weight_grad_workspace(int(M), int(Ca), int(Cz), int(dtype), int(fmt), _device_index(device),
                                  os.environ.get("DROPIT_WG_PATH", ""))


def dropit_weight_grad(dy: torch.Tensor, cache: DropITCache, out: Optional[torch.Tensor] = None,
                       accumulate: bool = False, workspace: Optional[torch.Tensor] = None,
                       fused: bool = False) -> torch.Tensor:
    """Eq. 6: dW[j, c] = sum over retained (n, c) of dY[n, j] a[n, c]; returns fp32 [Cz, Ca].

    fused=True calls dropit_weight_grad_fused (cache expanded inside the GEMM, no dense scratch)."""
    cache = dropit_dequantize_cache(cache)
    _require_cuda(dy, "dy")
    if dy.dtype != cache.dtype:
        raise TypeError("dy dtype %s != cache dtype %s" % (dy.dtype, cache.dtype))
    Ca = cache.shape[-1]
    M = cache.n // Ca if Ca else 0
    Cz = dy.shape[-1]
    if dy.numel() != M * Cz:
        raise ValueError("dy has %d elements, expected %d x %d" % (dy.numel(), M, Cz))
    lib = _lib.load()
    dev = dy.device
    dt = _DTYPE_CODE[cache.dtype]
    if out is None:
        if accumulate:
            raise ValueError("accumulate=True needs out")
        out = torch.empty((Cz, Ca), dtype=torch.float32, device=dev)
    wb = dropit_weight_grad_workspace(M, Ca, Cz, dt, cache.fmt, dev)
    if workspace is None or workspace.numel() < wb:
        workspace = torch.empty(max(wb, 16), dtype=torch.uint8, device=dev)
    with _on_device(dev):
        fn = lib.dropit_weight_grad_fused if fused else lib.dropit_weight_grad
        code = fn(_ptr(dy), _ptr(cache.values), _ptr(cache.meta), _ptr(cache.offsets), M, Ca, Cz,
                                      cache.k, dt, cache.fmt, _ptr(out), int(bool(accumulate)), _ptr(workspace),
                                      workspace.numel(), _ptr(_status_word(dev)), _stream_ptr(dev))
    _check(code, "dropit_weight_grad_fused" if fused else "dropit_weight_grad")
    return out


@functools.lru_cache(maxsize=4096)
def _conv_weight_grad_workspace(B, Ca, H, W, Cz, R, S, stride, pad, dtype: int, fmt: int, dev_index: int) -> int:
    out = ctypes.c_size_t(0)
    with _on_device(torch.device("cuda", dev_index)):
        code = _lib.load().dropit_conv_weight_grad_workspace(B, Ca, H, W, Cz, R, S, stride, pad, dtype, fmt,
                                                             ctypes.byref(out))
    _check(code, "dropit_conv_weight_grad_workspace")
    return int(out.value)


def dropit_conv_weight_grad_workspace(B, Ca, H, W, Cz, R, S, stride, pad, dtype: int, fmt: int, device=None) -> int:
    """Scratch bytes of dropit_conv_weight_grad on `device` (the split count depends on its SM count)."""
    return _conv_weight_grad_workspace(B, Ca, H, W, Cz, R, S, stride, pad, int(dtype), int(fmt), _device_index(device))


def dropit_conv_weight_grad(dy: torch.Tensor, cache: DropITCache, kernel_size: Tuple[int, int], stride: int = 1,
                            pad: int = 0, dilation: int = 1, out: Optional[torch.Tensor] = None,
                            accumulate: bool = False, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Eq. 4-5 retained term: dW[j,c,u,v] from dY [B,Cz,Ho,Wo] and the cache of a [B,Ca,H,W]; fp32."""
    cache = dropit_dequantize_cache(cache)
    _require_cuda(dy, "dy")
    if dy.dtype != cache.dtype:
        raise TypeError("dy dtype %s != cache dtype %s" % (dy.dtype, cache.dtype))
    B, Ca, H, W = cache.shape
    R, S = kernel_size
    Cz = dy.shape[1]
    lib = _lib.load()
    dev = dy.device
    dt = _DTYPE_CODE[cache.dtype]
    if out is None:
        if accumulate:
            raise ValueError("accumulate=True needs out")
        out = torch.empty((Cz, Ca, R, S), dtype=torch.float32, device=dev)
    wb = dropit_conv_weight_grad_workspace(B, Ca, H, W, Cz, R, S, stride, pad, dt, cache.fmt, dev)
    if workspace is None or workspace.numel() < wb:
        workspace = torch.empty(max(wb, 16), dtype=torch.uint8, device=dev)
    with _on_device(dev):
        code = lib.dropit_conv_weight_grad(_ptr(dy), _ptr(cache.values), _ptr(cache.meta), _ptr(cache.offsets), B, Ca,
                                           H, W, Cz, R, S, stride, pad, dilation, cache.k, dt, cache.fmt, _ptr(out),
                                           int(bool(accumulate)), _ptr(workspace), workspace.numel(),
                                           _ptr(_status_word(dev)), _stream_ptr(dev))
    _check(code, "dropit_conv_weight_grad")
    return out
