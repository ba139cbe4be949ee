"""Seeded synthetic inputs shaped like the paper's CIFAR-10 layers.  This module is the only code
shared by the tests' CPU checker and the CUDA path: it draws values and permutes layouts, and holds
none of the method's arithmetic.

Recipe: tensors are drawn on the host in logical order (X as [N,C,H,W], dY as [N,K,P,Q]) in fp32
from torch.Generator(seed), seed = 190805460 + 100000*config + 100*layer_index + t (t = 0 for X,
1 for dY); X = max(N(0,1), 0) (or U(-1,1) for a raw-image input), dY = dy_std * N(0,1); then rounded
to bf16 (nearest even) where asked.  The same rounded values go to every consumer."""
from __future__ import annotations

import torch

from .layers import ConvLayer

BASE_SEED = 190805460


def seed_for(config: int, layer_index: int, t: int) -> int:
    return BASE_SEED + 100000 * config + 100 * layer_index + t


def make_x(layer: ConvLayer, dtype: torch.dtype, seed: int) -> torch.Tensor:
    """X in logical [N,C,H,W] order, host memory, `dtype` (torch.float32 or torch.bfloat16)."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    shape = (layer.n, layer.c, layer.h, layer.w)
    if layer.x_dist == "relu_normal":
        x = torch.randn(shape, generator=g, dtype=torch.float32).clamp_(min=0.0)
    elif layer.x_dist == "uniform_pm1":
        x = torch.rand(shape, generator=g, dtype=torch.float32).mul_(2.0).sub_(1.0)
    else:
        raise ValueError(layer.x_dist)
    return x.to(dtype)


def make_dy(layer: ConvLayer, dtype: torch.dtype, seed: int) -> torch.Tensor:
    """dY in logical [N,K,P,Q] order, host memory."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    dy = torch.randn((layer.n, layer.k, layer.p, layer.q), generator=g, dtype=torch.float32)
    return dy.mul_(layer.dy_std).to(dtype)


def make_layer_inputs(layer: ConvLayer, dtype: torch.dtype, config: int = 0, layer_index: int = 0):
    """(X [N,C,H,W], dY [N,K,P,Q]) for one layer of one workload."""
    return (make_x(layer, dtype, seed_for(config, layer_index, 0)),
            make_dy(layer, dtype, seed_for(config, layer_index, 1)))


def to_nhwc(x_nchw: torch.Tensor) -> torch.Tensor:
    """Contiguous [N,H,W,C] copy of a logical [N,C,H,W] tensor (pure data movement)."""
    return x_nchw.permute(0, 2, 3, 1).contiguous()


def krsc_to_kcrs(dw_krsc: torch.Tensor) -> torch.Tensor:
    """Logical [K,C,R,S] view of a [K,R,S,C] buffer (pure data movement)."""
    return dw_krsc.permute(0, 3, 1, 2)
