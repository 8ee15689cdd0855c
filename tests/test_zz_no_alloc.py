"""dropit_compress_static: the variant of dropit_compress that needs no workspace from the caller.

It serves callers that cannot allocate device memory when they compress (a runtime whose memory plan was
frozen beforehand, a plug-in that may not touch its host's allocator); its scratch is a fixed array
inside the library.  The test drives it through the C ABI and requires bit-identical caches to the
regular entry point, on two calls in a row so that what the first call leaves in the shared scratch
is shown not to disturb the second.  This file sorts last on purpose: a run that stops at the first
failure has then already run every other test.
"""
import ctypes

import pytest
import torch

import dropit_inputs as di
import paper_2202_13808_b200 as dropit
from paper_2202_13808_b200 import _lib

pytestmark = pytest.mark.gpu


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr() if t.numel() else 0)


def _compress_static(lib, x, gamma, fmt_code, status):
    """Call the C entry point directly; every buffer is allocated by the test beforehand."""
    n = x.numel()
    vb, mb, ob, _ = dropit.dropit_cache_sizes(n, gamma, dropit.BF16, fmt_code)
    values = torch.empty(vb // 2, dtype=torch.bfloat16, device=x.device)
    meta = torch.empty(mb // 4, dtype=torch.int32, device=x.device)
    offsets = torch.empty(ob // 4, dtype=torch.int32, device=x.device)
    stream = ctypes.c_void_p(torch.cuda.current_stream(x.device).cuda_stream)
    code = lib.dropit_compress_static(_ptr(x), n, float(gamma), fmt_code, _ptr(values), _ptr(meta), _ptr(offsets),
                                      _ptr(status), stream)
    return code, values, meta, offsets


def test_static_scratch_variant_matches_the_regular_entry_point_twice_in_a_row(cuda_device):
    lib = _lib.load()
    assert 0 < lib.dropit_compress_static_scratch_bytes() < (1 << 20)
    status = torch.zeros(4, dtype=torch.int32, device=cuda_device)
    cases = [
        (di.small_linear(3000, 768, 1, "bf16", 0.9), 0.9, "bitmask"),          # sampled band, several blocks per warp
        (di.small_conv(3, 64, 56, 56, 1, 1, 1, gamma=0.8), 0.8, "bitmask"),     # post-ReLU ties, other size and gamma
        (di.small_linear(257, 129, 1, "bf16", 0.5), 0.5, "index32"),            # small ragged tensor, general path
        (di.small_linear(3000, 768, 1, "bf16", 0.9), 0.9, "bitmask"),          # first input again after the others
    ]
    for case, gamma, fmt in cases:
        x = di.make_x(case).to(cuda_device)
        fmt_code = dropit.FMT_BITMASK if fmt == "bitmask" else dropit.FMT_INDEX32
        ref = dropit.dropit_compress(x, gamma, fmt)
        for _ in range(2):   # two calls in a row share the built-in scratch
            code, values, meta, offsets = _compress_static(lib, x, gamma, fmt_code, status)
            assert code == 0, dropit.dropit_status_string(code)
            torch.cuda.synchronize(cuda_device)
            assert int(status[0].item()) == 0
            assert torch.equal(values.view(torch.int16), ref.values.view(torch.int16))
            assert torch.equal(meta, ref.meta)
            assert torch.equal(offsets, ref.offsets)
    dropit.check_device_status(cuda_device)


def test_static_scratch_variant_allocates_no_device_memory(cuda_device):
    """With every buffer in place beforehand, the call itself must leave the device's memory as it was: nothing
    taken from the driver (free bytes as the driver reports them) and nothing from torch's allocator."""
    lib = _lib.load()
    case = di.small_linear(3000, 768, 1, "bf16", 0.9)
    x = di.make_x(case).to(cuda_device)
    n = x.numel()
    vb, mb, ob, _ = dropit.dropit_cache_sizes(n, 0.9, dropit.BF16, dropit.FMT_BITMASK)
    values = torch.empty(vb // 2, dtype=torch.bfloat16, device=cuda_device)
    meta = torch.empty(mb // 4, dtype=torch.int32, device=cuda_device)
    offsets = torch.empty(ob // 4, dtype=torch.int32, device=cuda_device)
    status = torch.zeros(4, dtype=torch.int32, device=cuda_device)
    stream = ctypes.c_void_p(torch.cuda.current_stream(cuda_device).cuda_stream)

    def call():
        return lib.dropit_compress_static(_ptr(x), n, 0.9, dropit.FMT_BITMASK, _ptr(values), _ptr(meta), _ptr(offsets),
                                          _ptr(status), stream)

    assert call() == 0          # the first call on a device looks up the scratch address and sets kernel attributes
    torch.cuda.synchronize(cuda_device)
    free0, _ = torch.cuda.mem_get_info(cuda_device)
    alloc0, reserved0 = torch.cuda.memory_allocated(cuda_device), torch.cuda.memory_reserved(cuda_device)
    for _ in range(3):
        assert call() == 0
    torch.cuda.synchronize(cuda_device)
    free1, _ = torch.cuda.mem_get_info(cuda_device)
    assert free0 - free1 < (1 << 20)      # (device-wide figure: allow for noise below one allocation granule)
    assert torch.cuda.memory_allocated(cuda_device) == alloc0 and torch.cuda.memory_reserved(cuda_device) == reserved0
    assert int(status[0].item()) == 0


def test_static_scratch_variant_rejects_oversize_and_bad_arguments(cuda_device):
    lib = _lib.load()
    null = ctypes.c_void_p(0)
    a16 = ctypes.c_void_p(16)
    # larger than the stated maximum: refused before anything is launched
    assert lib.dropit_compress_static(a16, (1 << 28) + 1, 0.5, 0, a16, a16, a16, null, null) == 3
    assert lib.dropit_compress_static(null, 100, 0.5, 0, a16, a16, a16, null, null) == 1
    assert lib.dropit_compress_static(a16, 100, 1.5, 0, a16, a16, a16, null, null) == 1
    assert lib.dropit_compress_static(null, 0, 0.5, 0, null, null, null, null, null) == 0
