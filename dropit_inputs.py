"""Seeded synthetic layer inputs shaped like the DropIT paper's workloads.

This module only draws random tensors (CPU `torch.Generator`, fp32 draw, then a
cast); it holds none of DropIT's arithmetic and serves the CPU oracle's tests,
the GPU parity tests and the benchmark alike.  The tensors stand in for the
activations of DeiT / ViT-B/16 / ResNet / R-CNN on ImageNet, CIFAR-100 and COCO
(Sec. 4 of arXiv 2202.13808), which are not shipped: post-LayerNorm inputs are
N(0,1), MLP fc2 inputs are GELU(N(0,1)), conv inputs are ReLU(N(0,1)) (about
half exact zeros, so heavy ties), incoming gradients are N(0, 0.02^2).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

_DTYPES = {"bf16": torch.bfloat16, "f32": torch.float32}


@dataclass(frozen=True)
class LinearCase:
    """One fully-connected layer call: a [M, Ca] -> z [M, Cz]."""
    name: str
    M: int
    Ca: int
    Cz: int
    dtype: str = "bf16"
    gamma: float = 0.9
    x_dist: str = "normal"   # normal | gelu | relu
    dy_std: float = 0.02

    @property
    def n(self) -> int:
        return self.M * self.Ca

    @property
    def torch_dtype(self):
        return _DTYPES[self.dtype]


@dataclass(frozen=True)
class ConvCase:
    """One Conv2d layer call: a [B, Ca, H, W] (NCHW) -> z [B, Cz, Ho, Wo]."""
    name: str
    B: int
    Ca: int
    H: int
    W: int
    Cz: int
    R: int
    S: int
    stride: int = 1
    pad: int = 0
    dtype: str = "bf16"
    gamma: float = 0.8
    x_dist: str = "relu"
    dy_std: float = 0.02

    @property
    def n(self) -> int:
        return self.B * self.Ca * self.H * self.W

    @property
    def Ho(self) -> int:
        return (self.H + 2 * self.pad - self.R) // self.stride + 1

    @property
    def Wo(self) -> int:
        return (self.W + 2 * self.pad - self.S) // self.stride + 1

    @property
    def torch_dtype(self):
        return _DTYPES[self.dtype]


# The layer calls of the evaluation configurations.
SINGLE_LINEAR_F32 = LinearCase("linear_f32_256x768", 256, 768, 768, dtype="f32", gamma=0.9, dy_std=1.0)
VITB_FC1 = LinearCase("vitb_fc1", 64 * 197, 768, 3072, gamma=0.9)
VITB_FC2 = LinearCase("vitb_fc2", 64 * 197, 3072, 768, gamma=0.9, x_dist="gelu")
R50_CONV1X1 = ConvCase("r50_conv1x1", 64, 256, 56, 56, 64, 1, 1, pad=0, gamma=0.8)
R50_CONV3X3 = ConvCase("r50_conv3x3", 64, 64, 56, 56, 64, 3, 3, pad=1, gamma=0.8)
VITDET_QKV = LinearCase("vitdet_qkv", 8 * 4096, 768, 2304, gamma=0.9)
VITDET_FC1 = LinearCase("vitdet_fc1", 8 * 4096, 768, 3072, gamma=0.9)
VITDET_FC2 = LinearCase("vitdet_fc2", 8 * 4096, 3072, 768, gamma=0.9, x_dist="gelu")


def with_gamma(case, gamma: float):
    return replace(case, gamma=gamma, name="%s_g%g" % (case.name, gamma))


def _draw(shape, seed: int, dist: str, std: float, dtype) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    t = torch.randn(shape, generator=g, dtype=torch.float32)
    if dist == "gelu":
        t = torch.nn.functional.gelu(t)
    elif dist == "relu":
        t = torch.relu(t)
    elif dist != "normal":
        raise ValueError(dist)
    if std != 1.0:
        t = t * std
    return t.to(dtype).contiguous()


def make_x(case, batch: int = 0) -> torch.Tensor:
    """The layer input a (CPU tensor). `batch` picks an independent draw."""
    if isinstance(case, LinearCase):
        shape = (case.M, case.Ca)
    else:
        shape = (case.B, case.Ca, case.H, case.W)
    return _draw(shape, 2 * batch, case.x_dist, 1.0, case.torch_dtype)


def make_dy(case, batch: int = 0) -> torch.Tensor:
    """The incoming gradient of the layer output (CPU tensor)."""
    if isinstance(case, LinearCase):
        shape = (case.M, case.Cz)
    else:
        shape = (case.B, case.Cz, case.Ho, case.Wo)
    return _draw(shape, 2 * batch + 1, "normal", case.dy_std, case.torch_dtype)


def small_linear(M, Ca, Cz, dtype="bf16", gamma=0.9, x_dist="normal", dy_std=0.02) -> LinearCase:
    return LinearCase("lin_%dx%dx%d_%s_g%g_%s" % (M, Ca, Cz, dtype, gamma, x_dist), M, Ca, Cz, dtype, gamma, x_dist,
                      dy_std)


def small_conv(B, Ca, H, W, Cz, R, S, stride=1, pad=0, dtype="bf16", gamma=0.8, x_dist="relu") -> ConvCase:
    return ConvCase("conv_%dx%dx%dx%d_%d_%dx%d_s%dp%d_%s_g%g" % (B, Ca, H, W, Cz, R, S, stride, pad, dtype, gamma),
                    B, Ca, H, W, Cz, R, S, stride, pad, dtype, gamma, x_dist)
