"""Shared helpers of the parity tests: run the CUDA path through the binding, run the oracle on the
same values, and compare with the normalised error metric."""
from __future__ import annotations

import numpy as np
import torch

from oracle import oracle
from paper_1908_05460_b200 import binding as B
from paper_1908_05460_b200 import inputs as I
from paper_1908_05460_b200.layers import ConvLayer

TOL_F32 = 1e-5     # fp32 paths: max |gpu - oracle| / sum|products|
TOL_BF16 = 2e-2    # bf16 tensor-core paths
TOL_SUM = 1e-6     # selection sums, relative to sum |dY[n,k,:,:]|


def oshape(l: ConvLayer) -> oracle.Shape:
    return oracle.Shape(l.n, l.c, l.h, l.w, l.k, l.r, l.s, l.stride, l.stride, l.pad, l.pad)


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float64).numpy()


class GpuLayer:
    """Device buffers + descriptor of one layer in the library's layouts."""

    def __init__(self, layer: ConvLayer, dtype, x_nchw: torch.Tensor, dy: torch.Tensor, *, x_layout=B.X_NHWC,
                 dw_layout=B.DW_KRSC, alpha=1.0, rand_std=1.0 / 128, algo=B.ALGO_AUTO, math=B.MATH_DEFAULT, topk=1,
                 dy_layout=B.DY_NKPQ, sm_budget=0):
        self.layer, self.dtype, self.dw_layout = layer, dtype, dw_layout
        self.x = (I.to_nhwc(x_nchw) if x_layout == B.X_NHWC else x_nchw.contiguous()).cuda()
        self.dy = (dy.contiguous() if dy_layout == B.DY_NKPQ else dy.permute(0, 2, 3, 1).contiguous()).cuda()
        shape = {B.DW_KRSC: (layer.k, layer.r, layer.s, layer.c), B.DW_KCRS: (layer.k, layer.c, layer.r, layer.s),
                 B.DW_RSCK: (layer.r, layer.s, layer.c, layer.k)}[dw_layout]
        self.dw = torch.full(shape, float("nan"), dtype=torch.float32, device="cuda")
        self.desc = B.make_desc(layer, dtype, x_layout=x_layout, dw_layout=dw_layout, alpha=alpha, rand_std=rand_std,
                                algo=algo, math=math, topk=topk, dy_layout=dy_layout, sm_budget=sm_budget)
        self.ws = B.attach_workspace(self.desc)

    def logical_dw(self) -> np.ndarray:
        torch.cuda.synchronize()
        d = self.dw.cpu()
        if self.dw_layout == B.DW_KRSC:
            d = I.krsc_to_kcrs(d)
        elif self.dw_layout == B.DW_RSCK:
            d = d.permute(3, 2, 0, 1).contiguous()
        return d.to(torch.float64).numpy()

    def exact(self):
        self.dw.fill_(float("nan"))
        B.gaconv_dw_exact(self.x, self.dy, self.dw, self.desc)
        return self.logical_dw()

    def approx(self, method, seed=0):
        self.dw.fill_(float("nan"))
        B.gaconv_dw_approx(method, self.x, self.dy, self.dw, self.desc, seed)
        return self.logical_dw()

    def select_topk(self):
        l = self.layer
        t = min(self.desc.topk, l.p * l.q)
        idx = torch.full((l.n, l.k, t), -1, dtype=torch.int32, device="cuda")
        s = torch.full((l.n, l.k), float("nan"), dtype=torch.float32, device="cuda")
        B.gaconv_approx_select_topk(self.dy, idx, s, self.desc)
        torch.cuda.synchronize()
        return idx.cpu().numpy(), s.cpu().numpy().astype(np.float64)

    def select(self, want_sparse=False):
        l = self.layer
        idx = torch.full((l.n, l.k), -1, dtype=torch.int32, device="cuda")
        s = torch.full((l.n, l.k), float("nan"), dtype=torch.float32, device="cuda")
        sp = torch.full_like(self.dy, float("nan")) if want_sparse else None
        B.gaconv_approx_select(self.dy, idx, s, sp, self.desc)
        torch.cuda.synchronize()
        return idx.cpu().numpy(), s.cpu().numpy().astype(np.float64), (None if sp is None else sp.cpu())


def norm_err(gpu: np.ndarray, ref: np.ndarray, dnorm: np.ndarray) -> float:
    """max over elements of |gpu - ref| / dnorm; where dnorm == 0 the gpu value must be exactly 0."""
    assert gpu.shape == ref.shape == dnorm.shape
    assert np.all(np.isfinite(gpu)), "non-finite output (unwritten element?)"
    zero = dnorm == 0
    assert np.all(gpu[zero] == 0), "non-zero output where every product is zero"
    if np.all(zero):
        return 0.0
    return float(np.max(np.abs(gpu - ref)[~zero] / dnorm[~zero]))
