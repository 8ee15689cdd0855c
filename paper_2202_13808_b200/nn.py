"""torch.autograd wrappers: Linear and Conv2d layers that cache D(a) instead of a (Sec. 3.2, Fig. 1b).

Forward: z = l(a, theta) by the stock kernel (DropIT does not touch the forward pass, Sec. 3.5), then
the layer input is compressed with `dropit_compress` and only {values, mask/indices, seek table} are
saved for backward, so the dense input's last reference can die and the caching allocator gets its
bytes back before the next layer allocates (App. A.6).
Backward: the weight gradient comes from the compressed cache (Eq. 4-6); the input gradient and the
bias gradient need theta / dY only (Eq. 3) and use stock torch.

Applies to fully-connected and convolutional layers only; normalisation and activation layers keep
their caches (Sec. 3.5).
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.nn as nn
import torch.nn.functional as F

from . import api


def _compress(x: torch.Tensor, gamma: float, fmt: str, seed):
    """Min-k (seed None) or random (an integer seed) compression of a layer input: the two strategies of Sec. 3.3."""
    if seed is None:
        return api.dropit_compress(x, gamma, fmt)
    return api.dropit_compress_random(x, gamma, int(seed), fmt)


def _cache_dtype(x: torch.Tensor, weight: torch.Tensor) -> torch.dtype:
    """The dtype the layer's matmul really runs in, which is the dtype its input is cached in: under autocast
    the autocast dtype, otherwise the weight's.  (An fp32 activation in front of bf16 weights would otherwise be
    cached in fp32 and take the fp32 kernels, three times the cache and no tensor cores.)  Anything but bf16
    falls back to the input's own dtype."""
    dt = torch.get_autocast_dtype("cuda") if torch.is_autocast_enabled("cuda") else weight.dtype
    return torch.bfloat16 if dt == torch.bfloat16 else x.dtype


def _check_input(x: torch.Tensor):
    if not x.is_cuda:
        raise ValueError("DropIT layers need CUDA tensors (there is no CPU path)")
    if x.dtype not in (torch.bfloat16, torch.float32):
        raise TypeError("DropIT layers take bf16 or fp32 activations, got %s" % x.dtype)


class DropITLinearFn(torch.autograd.Function):
    """y = x W^T + b with the cached x replaced by its min-k compression."""

    @staticmethod
    def forward(ctx, x, weight, bias, gamma: float, fmt: str, seed=None, quant: bool = False):
        _check_input(x)
        z = F.linear(x, weight, bias)
        ctx.has_bias = bias is not None
        ctx.bias_dtype = bias.dtype if bias is not None else None
        ctx.x_shape, ctx.x_dtype = tuple(x.shape), x.dtype
        ctx.cache_meta = None
        if weight.requires_grad:
            x2 = x.reshape(-1, x.shape[-1])
            if x2.dtype != _cache_dtype(x2, weight):
                x2 = x2.to(torch.bfloat16)
            if not x2.is_contiguous():
                x2 = x2.contiguous()
            cache = _compress(x2, gamma, fmt, seed)
            ctx.cache_meta = (cache.n, cache.k, cache.shape, cache.dtype, cache.fmt, cache.gamma)
            ctx.quant = bool(quant) and cache.dtype == torch.bfloat16
            if ctx.quant:   # the retained values as 8-bit codes: 1 byte per retained element
                cache = api.dropit_quantize_cache(cache)
                ctx.save_for_backward(weight, cache.codes, cache.meta, cache.offsets, cache.scale)
            else:
                ctx.save_for_backward(weight, cache.values, cache.meta, cache.offsets)
        else:
            ctx.save_for_backward(weight)
        return z

    @staticmethod
    def backward(ctx, dz):
        saved = ctx.saved_tensors
        weight = saved[0]
        dx = dw = db = None
        dz2 = dz.reshape(-1, dz.shape[-1])
        if ctx.needs_input_grad[0]:
            dx = (dz2 @ weight.to(dz2.dtype)).reshape(ctx.x_shape).to(ctx.x_dtype)   # Eq. 3: exact, needs theta only
        if ctx.needs_input_grad[1] and ctx.cache_meta is not None:
            n, k, shape, dtype, fmt, gamma = ctx.cache_meta
            if ctx.quant:
                cache = api.DropITCache(None, saved[2], saved[3], n, k, shape, dtype, fmt, gamma, saved[1], saved[4])
            else:
                cache = api.DropITCache(saved[1], saved[2], saved[3], n, k, shape, dtype, fmt, gamma)
            dzc = dz2 if dz2.is_contiguous() else dz2.contiguous()
            if dzc.dtype != dtype:
                dzc = dzc.to(dtype)
            dw = api.dropit_weight_grad(dzc, cache).to(weight.dtype)   # Eq. 6
        if ctx.has_bias and ctx.needs_input_grad[2]:
            db = dz2.sum(0).to(ctx.bias_dtype)
        return dx, dw, db, None, None, None, None


class DropITConv2dFn(torch.autograd.Function):
    """Conv2d (groups 1, dilation 1) with the cached input replaced by its min-k compression."""

    @staticmethod
    def forward(ctx, x, weight, bias, stride: int, padding: int, gamma: float, fmt: str, seed=None):
        _check_input(x)
        z = F.conv2d(x, weight, bias, stride=stride, padding=padding)
        ctx.has_bias = bias is not None
        ctx.x_shape = tuple(x.shape)
        ctx.stride, ctx.padding = stride, padding
        ctx.cache_meta = None
        if weight.requires_grad:
            xc = x if x.dtype == _cache_dtype(x, weight) else x.to(torch.bfloat16)
            xc = xc if xc.is_contiguous() else xc.contiguous()
            cache = _compress(xc, gamma, fmt, seed)
            ctx.cache_meta = (cache.n, cache.k, cache.shape, cache.dtype, cache.fmt, cache.gamma)
            ctx.save_for_backward(weight, cache.values, cache.meta, cache.offsets)
        else:
            ctx.save_for_backward(weight)
        return z

    @staticmethod
    def backward(ctx, dz):
        saved = ctx.saved_tensors
        weight = saved[0]
        dx = dw = db = None
        if ctx.needs_input_grad[0]:
            dx = torch.nn.grad.conv2d_input(ctx.x_shape, weight, dz, stride=ctx.stride, padding=ctx.padding)
        if ctx.needs_input_grad[1] and ctx.cache_meta is not None:
            n, k, shape, dtype, fmt, gamma = ctx.cache_meta
            cache = api.DropITCache(saved[1], saved[2], saved[3], n, k, shape, dtype, fmt, gamma)
            dzc = dz if dz.is_contiguous() else dz.contiguous()
            if dzc.dtype != dtype:
                dzc = dzc.to(dtype)
            dw = api.dropit_conv_weight_grad(dzc, cache, (weight.shape[2], weight.shape[3]), ctx.stride,
                                             ctx.padding).to(weight.dtype)   # Eq. 4-5
        if ctx.has_bias and ctx.needs_input_grad[2]:
            db = dz.sum((0, 2, 3))
        return dx, dw, db, None, None, None, None, None


class DropITGeluLinearFn(torch.autograd.Function):
    """z = GELU(x) W^T + b for bf16 tensors, with the GELU written by the library's producer kernel so that the
    selection statistics of GELU(x), the tensor the Linear caches, are taken while it is written (Sec. 3.5: the
    activation keeps its own cache x; only the Linear's cache is replaced by D(GELU(x)))."""

    @staticmethod
    def forward(ctx, x, weight, bias, gamma: float, fmt: str):
        _check_input(x)
        x2 = x.reshape(-1, x.shape[-1])
        x2 = x2 if x2.is_contiguous() else x2.contiguous()
        y, prep = api.dropit_produce(x2, gamma, "gelu")
        z = F.linear(y, weight, bias).reshape(*x.shape[:-1], weight.shape[0])
        ctx.has_bias = bias is not None
        ctx.x_shape = tuple(x.shape)
        cache = api.dropit_compress_prepared(y, gamma, prep, fmt)
        ctx.cache_meta = (cache.n, cache.k, cache.shape, cache.dtype, cache.fmt, cache.gamma)
        ctx.save_for_backward(x2, weight, cache.values, cache.meta, cache.offsets)
        return z

    @staticmethod
    def backward(ctx, dz):
        x2, weight, values, meta, offsets = ctx.saved_tensors
        dx = dw = db = None
        dz2 = dz.reshape(-1, dz.shape[-1])
        if ctx.needs_input_grad[0]:
            dy = dz2 @ weight                                             # Eq. 3: exact, needs theta only
            dx = torch.ops.aten.gelu_backward(dy, x2).reshape(ctx.x_shape)   # the activation's own cache is x
        if ctx.needs_input_grad[1]:
            n, k, shape, dtype, fmt, gamma = ctx.cache_meta
            cache = api.DropITCache(values, meta, offsets, n, k, shape, dtype, fmt, gamma)
            dzc = dz2 if dz2.is_contiguous() else dz2.contiguous()
            dw = api.dropit_weight_grad(dzc.to(dtype), cache).to(weight.dtype)   # Eq. 6
        if ctx.has_bias and ctx.needs_input_grad[2]:
            db = dz2.sum(0)
        return dx, dw, db, None, None


class _Strategy:
    """Dropping strategy of a layer (Sec. 3.3): "min_k", or "random" with a seed that advances by one per call."""

    def _init_strategy(self, strategy: str, seed: int):
        if strategy not in ("min_k", "random"):
            raise ValueError("strategy must be 'min_k' or 'random'")
        self.strategy, self.seed, self._calls = strategy, int(seed), 0

    def _next_seed(self):
        if self.strategy == "min_k":
            return None
        self._calls += 1
        return self.seed + self._calls - 1


class DropITLinear(nn.Linear, _Strategy):
    """nn.Linear whose backward uses a compressed input cache. `gamma` is the dropped fraction."""

    def __init__(self, in_features, out_features, bias=True, gamma: float = 0.9, fmt: str = "bitmask",
                 strategy: str = "min_k", seed: int = 0, quantize: bool = False, **kw):
        super().__init__(in_features, out_features, bias=bias, **kw)
        self.gamma, self.fmt = float(gamma), fmt
        self.quantize = bool(quantize)     # keep the retained values as 8-bit codes (bf16 activations only)
        self._init_strategy(strategy, seed)

    def forward(self, x):
        if not (self.training and torch.is_grad_enabled()):
            return F.linear(x, self.weight, self.bias)     # inference is unchanged (Sec. 3.5)
        return DropITLinearFn.apply(x, self.weight, self.bias, self.gamma, self.fmt, self._next_seed(), self.quantize)


class DropITGeluLinear(nn.Linear):
    """GELU followed by nn.Linear (an MLP's second layer together with the activation in front of it), bf16, with the
    Linear's input cache compressed from statistics that the GELU kernel takes on the way."""

    def __init__(self, in_features, out_features, bias=True, gamma: float = 0.9, fmt: str = "bitmask", **kw):
        super().__init__(in_features, out_features, bias=bias, **kw)
        self.gamma, self.fmt = float(gamma), fmt

    def forward(self, x):
        if not (self.training and torch.is_grad_enabled()) or x.dtype != torch.bfloat16:
            return F.linear(F.gelu(x), self.weight, self.bias)
        return DropITGeluLinearFn.apply(x, self.weight, self.bias, self.gamma, self.fmt)


class DropITConv2d(nn.Conv2d, _Strategy):
    """nn.Conv2d (groups 1, dilation 1, square stride/padding) with a compressed input cache."""

    def __init__(self, *args, gamma: float = 0.8, fmt: str = "bitmask", strategy: str = "min_k", seed: int = 0, **kw):
        super().__init__(*args, **kw)
        self._init_strategy(strategy, seed)
        if self.groups != 1 or self.dilation != (1, 1) or self.stride[0] != self.stride[1] or \
                self.padding[0] != self.padding[1] or self.padding_mode != "zeros":
            raise ValueError("DropITConv2d supports groups=1, dilation=1, square stride and zero padding")
        self.gamma, self.fmt = float(gamma), fmt

    def forward(self, x):
        if not (self.training and torch.is_grad_enabled()):
            return F.conv2d(x, self.weight, self.bias, self.stride, self.padding)
        return DropITConv2dFn.apply(x, self.weight, self.bias, self.stride[0], self.padding[0], self.gamma, self.fmt,
                                    self._next_seed())


def convert_linear_layers(module: nn.Module, gamma: float, fmt: str = "bitmask",
                          skip: Optional[set] = None) -> nn.Module:
    """Replace every nn.Linear below `module` (except names in `skip`) by a DropITLinear sharing its parameters."""
    skip = skip or set()
    for name, child in list(module.named_children()):
        if isinstance(child, nn.Linear) and not isinstance(child, (DropITLinear, DropITGeluLinear)) and name not in skip:
            new = DropITLinear(child.in_features, child.out_features, bias=child.bias is not None, gamma=gamma, fmt=fmt,
                               device=child.weight.device, dtype=child.weight.dtype)
            new.weight, new.bias = child.weight, child.bias
            setattr(module, name, new)
        else:
            convert_linear_layers(child, gamma, fmt, skip)
    return module
