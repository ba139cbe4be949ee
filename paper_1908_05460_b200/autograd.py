"""Training-step integration: a convolution whose filter gradient comes from this library.

Forward and the input gradient stay with the framework (torch / cuDNN); only the filter gradient --
the operation the paper approximates, "roughly a third" of a layer's time (Section 2) -- is computed
by gaconv, exactly or by the method the approximation schedule picks for this layer at this training
step (Sections 2.5 and 3).  Weights and inputs are bf16 or fp32 CUDA tensors; the layer keeps its
activations in channels-last memory (the NHWC layout of the paper's kernel, Section 2.4), so the
library reads torch's buffers in place and writes the gradient straight in torch's [K,C,R,S] layout.
"""
from __future__ import annotations

import torch
import torch.nn.functional as F

from . import binding as B
from .layers import ConvLayer


class _Conv2dFilterGrad(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, weight, module):
        ctx.module = module
        ctx.save_for_backward(x, weight)
        return F.conv2d(x, weight, None, module.stride, module.padding)

    @staticmethod
    def backward(ctx, dy):
        x, weight = ctx.saved_tensors
        m = ctx.module
        dx = torch.nn.grad.conv2d_input(x.shape, weight, dy, m.stride, m.padding) if ctx.needs_input_grad[0] else None
        dw = m.filter_gradient(x, dy) if ctx.needs_input_grad[1] else None
        return dx, dw, None


class GAConv2d(torch.nn.Module):
    """3x3 / 5x5 / ... convolution (no bias, dilation 1, one group) with the library's filter gradient.

    `schedule` (binding.Schedule) and `layer_index` say which method this layer uses at `step`; advance
    `step` once per batch (`module.step += 1`, or share one counter object across layers).  Without a
    schedule the gradient is always exact."""

    def __init__(self, in_channels, out_channels, kernel_size, stride=1, padding=0, schedule=None, layer_index=0,
                 dtype=torch.float32, device="cuda"):
        super().__init__()
        self.stride, self.padding, self.kernel_size = stride, padding, kernel_size
        self.weight = torch.nn.Parameter(torch.empty(out_channels, in_channels, kernel_size, kernel_size, dtype=dtype, device=device))
        torch.nn.init.kaiming_normal_(self.weight)
        self.schedule, self.layer_index, self.step = schedule, layer_index, 0
        self._desc_cache = {}

    def forward(self, x):
        return _Conv2dFilterGrad.apply(x.contiguous(memory_format=torch.channels_last), self.weight, self)

    def _desc(self, x, dy_layout=B.DY_NKPQ):
        key = (tuple(x.shape), x.dtype, dy_layout)
        if key not in self._desc_cache:
            n, c, h, w = x.shape
            k = self.weight.shape[0]
            layer = ConvLayer("gaconv2d", n, c, h, w, k, self.kernel_size, self.kernel_size, self.stride, self.padding)
            d = B.make_desc(layer, x.dtype, x_layout=B.X_NHWC, dw_layout=B.DW_KCRS, alpha=1.0, dy_layout=dy_layout)
            self._desc_cache[key] = (d, B.attach_workspace(d, methods=(B.METHOD_EXACT, B.METHOD_TOP1), device=x.device))
        return self._desc_cache[key][0]

    def filter_gradient(self, x, dy):
        """dW [K,C,R,S] (the weight's dtype) of this layer for activations x and output gradient dy."""
        B.load()
        x = x.contiguous(memory_format=torch.channels_last)        # NHWC memory under an NCHW-shaped tensor
        if dy.dtype != x.dtype:
            dy = dy.to(x.dtype)
        # the gradient of a channels-last forward arrives channels-last: the library takes it as it is ([N,P,Q,K] memory)
        if dy.dim() == 4 and dy.shape[1] > 1 and not dy.is_contiguous() and dy.is_contiguous(memory_format=torch.channels_last):
            dy_layout = B.DY_NPQK
        else:
            dy, dy_layout = dy.contiguous(), B.DY_NKPQ             # [N,K,P,Q]
        dw = torch.empty(self.weight.shape, dtype=torch.float32, device=x.device)
        d = self._desc(x, dy_layout)
        if self.schedule is None:
            B.gaconv_dw_exact(x, dy, dw, d)
        else:
            self.schedule.run_layer(self.layer_index, self.step, x, dy, dw, d)
        return dw.to(self.weight.dtype)
