"""ctypes loader for libdropit.so.  Fails loudly: there is no fallback implementation."""
from __future__ import annotations

import ctypes
import os
import threading

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdropit.so")

_lock = threading.Lock()
_lib = None

c_i64, c_int, c_dbl, c_vp, c_sz = ctypes.c_int64, ctypes.c_int, ctypes.c_double, ctypes.c_void_p, ctypes.c_size_t
p_sz = ctypes.POINTER(ctypes.c_size_t)

# name -> (restype, argtypes); mirrors include/dropit.h
SIGNATURES = {
    "dropit_version": (c_int, []),
    "dropit_launch_count": (ctypes.c_uint64, []),
    "dropit_status_string": (ctypes.c_char_p, [c_int]),
    "dropit_keep_count": (c_i64, [c_i64, c_dbl]),
    "dropit_cache_sizes": (c_int, [c_i64, c_dbl, c_int, c_int, p_sz, p_sz, p_sz, p_sz]),
    "dropit_compress": (c_int, [c_vp, c_i64, c_dbl, c_int, c_int, c_vp, c_vp, c_vp, c_vp, c_sz, c_vp, c_vp]),
    "dropit_compress_random_workspace": (c_int, [c_i64, c_dbl, p_sz]),
    "dropit_compress_random": (c_int, [c_vp, c_i64, c_dbl, ctypes.c_uint64, c_int, c_int, c_vp, c_vp, c_vp, c_vp, c_sz,
                                       c_vp, c_vp]),
    "dropit_quantize_values": (c_int, [c_vp, c_i64, c_vp, c_vp, c_vp]),
    "dropit_dequantize_values": (c_int, [c_vp, c_vp, c_i64, c_vp, c_vp]),
    "dropit_activation_table": (c_int, [c_int, c_vp, c_vp]),
    "dropit_produce_workspace": (c_int, [c_i64, p_sz]),
    "dropit_produce": (c_int, [c_vp, c_i64, c_dbl, c_int, c_vp, c_vp, c_vp, c_sz, c_vp]),
    "dropit_compress_prepared": (c_int, [c_vp, c_i64, c_dbl, c_int, c_vp, c_vp, c_vp, c_vp, c_sz, c_vp, c_sz, c_vp, c_vp]),
    "dropit_compress_static_scratch_bytes": (c_sz, []),
    "dropit_compress_static": (c_int, [c_vp, c_i64, c_dbl, c_int, c_vp, c_vp, c_vp, c_vp, c_vp]),
    "dropit_decompress": (c_int, [c_vp, c_vp, c_vp, c_i64, c_i64, c_int, c_int, c_vp, c_vp]),
    "dropit_weight_grad_workspace": (c_int, [c_i64, c_i64, c_i64, c_int, c_int, p_sz]),
    "dropit_weight_grad": (c_int, [c_vp, c_vp, c_vp, c_vp, c_i64, c_i64, c_i64, c_i64, c_int, c_int, c_vp, c_int,
                                   c_vp, c_sz, c_vp, c_vp]),
    "dropit_weight_grad_fused": (c_int, [c_vp, c_vp, c_vp, c_vp, c_i64, c_i64, c_i64, c_i64, c_int, c_int, c_vp, c_int,
                                         c_vp, c_sz, c_vp, c_vp]),
    "dropit_conv_weight_grad_workspace": (c_int, [c_int] * 9 + [c_int, c_int, p_sz]),
    "dropit_conv_weight_grad": (c_int, [c_vp, c_vp, c_vp, c_vp] + [c_int] * 10 + [c_i64, c_int, c_int, c_vp, c_int,
                                        c_vp, c_sz, c_vp, c_vp]),
}


def load():
    """Load libdropit.so and declare every entry point; raises if the library is absent."""
    global _lib
    with _lock:
        if _lib is None:
            if not os.path.exists(LIB_PATH):
                raise RuntimeError(
                    "libdropit.so is not built (%s). Run `python -m paper_2202_13808_b200.build`; "
                    "there is no fallback path." % LIB_PATH)
            lib = ctypes.CDLL(LIB_PATH)
            for name, (res, args) in SIGNATURES.items():
                fn = getattr(lib, name)
                fn.restype = res
                fn.argtypes = args
            _lib = lib
    return _lib
