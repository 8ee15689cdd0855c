"""DropIT layer path for NVIDIA B200: min-k activation compression and weight gradients
from the compressed cache (arXiv 2202.13808), as hand-written sm_100a CUDA kernels behind a
C ABI (`include/dropit.h`), with a thin torch binding.

The CUDA library is loaded on first use; if it is missing or cannot be loaded the call raises.
There is no CPU or eager fallback.
"""
from .api import (  # noqa: F401
    BF16, F32, FMT_BITMASK, FMT_INDEX32, CHUNK, DropITCache, DropITError,
    dropit_cache_sizes, dropit_compress, dropit_compress_random, dropit_compress_random_workspace, dropit_conv_weight_grad, dropit_conv_weight_grad_workspace,
    dropit_decompress, dropit_keep_count, dropit_launch_count, dropit_status_string, dropit_version, dropit_weight_grad,
    dropit_weight_grad_workspace, check_device_status, library_path,
    dropit_activation_table, dropit_produce, dropit_produce_workspace, dropit_compress_prepared,
    dropit_quantize_cache, dropit_dequantize_cache,
)
from .nn import (  # noqa: F401
    DropITConv2d, DropITConv2dFn, DropITGeluLinear, DropITGeluLinearFn, DropITLinear, DropITLinearFn, convert_linear_layers,
)
