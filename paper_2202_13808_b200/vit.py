"""A plain ViT-B/16 (12 blocks, hidden 768, MLP 3072, 12 heads, 1000 classes) on synthetic images, used to
measure a full training step with DropIT on every Linear layer against the same model with stock layers
(Sec. 3.5: fully-connected layers of attention and MLP and the classifier; LayerNorm, GELU and attention
keep their caches; the patch-projection convolution is left dense, App. A.6).

  python -m paper_2202_13808_b200.vit --batch 64 --gamma 0.9 --steps 5

Everything that DropIT does not touch is stock torch (LayerNorm, GELU, scaled-dot-product attention,
cross entropy, SGD).
"""
from __future__ import annotations

import argparse
import json

import torch
import torch.nn as nn
import torch.nn.functional as F

from .nn import DropITGeluLinear, convert_linear_layers


class Block(nn.Module):
    def __init__(self, dim: int, heads: int, mlp: int):
        super().__init__()
        self.heads = heads
        self.norm1 = nn.LayerNorm(dim)
        self.qkv = nn.Linear(dim, 3 * dim)
        self.proj = nn.Linear(dim, dim)
        self.norm2 = nn.LayerNorm(dim)
        self.fc1 = nn.Linear(dim, mlp)
        self.fc2 = nn.Linear(mlp, dim)
        self.gelu_in_fc2 = False      # True when fc2 is a DropITGeluLinear, which applies the GELU itself

    def forward(self, x):
        B, L, C = x.shape
        qkv = self.qkv(self.norm1(x)).reshape(B, L, 3, self.heads, C // self.heads).permute(2, 0, 3, 1, 4)
        a = F.scaled_dot_product_attention(qkv[0], qkv[1], qkv[2])
        x = x + self.proj(a.transpose(1, 2).reshape(B, L, C))
        h = self.fc1(self.norm2(x))
        return x + (self.fc2(h) if self.gelu_in_fc2 else self.fc2(F.gelu(h)))


class ViT(nn.Module):
    def __init__(self, image=224, patch=16, dim=768, depth=12, heads=12, mlp=3072, classes=1000):
        super().__init__()
        self.patch_embed = nn.Conv2d(3, dim, patch, stride=patch)
        n = (image // patch) ** 2
        self.cls = nn.Parameter(torch.zeros(1, 1, dim))
        self.pos = nn.Parameter(torch.randn(1, n + 1, dim) * 0.02)
        self.blocks = nn.ModuleList([Block(dim, heads, mlp) for _ in range(depth)])
        self.norm = nn.LayerNorm(dim)
        self.head = nn.Linear(dim, classes)

    def forward(self, img):
        x = self.patch_embed(img).flatten(2).transpose(1, 2)
        x = torch.cat([self.cls.expand(x.shape[0], -1, -1), x], 1) + self.pos
        for b in self.blocks:
            x = b(x)
        return self.head(self.norm(x)[:, 0])


def build_vit_b16(gamma=None, device="cuda", dtype=torch.bfloat16, depth=12, seed=0, fuse_gelu=False) -> ViT:
    """Random-initialised ViT-B/16; gamma=None keeps stock layers, otherwise every nn.Linear becomes DropITLinear.
    fuse_gelu: the MLP's GELU and second Linear become one DropITGeluLinear (the GELU kernel takes the selection
    statistics of its output, the compression reads that output once)."""
    torch.manual_seed(seed)
    model = ViT(depth=depth).to(device=device, dtype=dtype)
    if gamma is not None:
        if fuse_gelu:
            for b in model.blocks:
                old = b.fc2
                new = DropITGeluLinear(old.in_features, old.out_features, gamma=gamma, device=old.weight.device,
                                       dtype=old.weight.dtype)
                new.weight, new.bias = old.weight, old.bias
                b.fc2, b.gelu_in_fc2 = new, True
        convert_linear_layers(model, gamma)
    return model.train()


def train_steps(model: nn.Module, batch: int, steps: int, warmup: int = 2, lr: float = 1e-3, seed: int = 0):
    """Run `steps` SGD steps on synthetic 224x224 images ~N(0,1) with random labels.
    Returns (samples/s, peak bytes allocated during a step beyond the resident state, last loss)."""
    dev = next(model.parameters()).device
    g = torch.Generator(device="cpu").manual_seed(seed)
    img = torch.randn(batch, 3, 224, 224, generator=g).to(dev, dtype=next(model.parameters()).dtype)
    lab = torch.randint(0, 1000, (batch,), generator=g).to(dev)
    opt = torch.optim.SGD(model.parameters(), lr=lr)

    def step():
        opt.zero_grad(set_to_none=True)
        loss = F.cross_entropy(model(img).float(), lab)
        loss.backward()
        opt.step()
        return loss

    for _ in range(warmup):
        step()
    torch.cuda.synchronize(dev)
    base = torch.cuda.memory_allocated(dev)
    torch.cuda.reset_peak_memory_stats(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        loss = step()
    e1.record()
    torch.cuda.synchronize(dev)
    peak = torch.cuda.max_memory_allocated(dev) - base
    return batch * steps / (e0.elapsed_time(e1) / 1e3), peak, float(loss.detach())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--gamma", type=float, default=0.9)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--depth", type=int, default=12)
    args = ap.parse_args()
    out = {}
    for name, gamma in (("dense", None), ("dropit", args.gamma)):
        model = build_vit_b16(gamma, depth=args.depth)
        sps, peak, loss = train_steps(model, args.batch, args.steps)
        out[name] = {"samples_per_s": sps, "peak_step_bytes": peak, "loss": loss}
        del model
        torch.cuda.empty_cache()
    out["config"] = {"model": "ViT-B/16", "batch": args.batch, "gamma": args.gamma, "dtype": "bf16", "depth": args.depth,
                     "data": "synthetic"}
    out["peak_ratio"] = out["dropit"]["peak_step_bytes"] / max(out["dense"]["peak_step_bytes"], 1)
    out["speed_ratio"] = out["dropit"]["samples_per_s"] / out["dense"]["samples_per_s"]
    print(json.dumps(out))


if __name__ == "__main__":
    main()
