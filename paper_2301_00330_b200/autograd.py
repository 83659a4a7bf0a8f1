"""A convolution layer whose backward pass is the filtered one (Sections 3.3-3.4: Eq. (grad_x), Eq. (grad_w)).

Forward: the convolution itself is torch's (it is not part of the filtered path), and the
activation stash is taken by gf_stash_forward instead of keeping x (Section 3.4).  Backward:
gf_backward gives g_W and g_X from the incoming g_y, the stash and W.  Only marshalling
happens here; every step of the path runs in the CUDA library.

Geometry: what the library accepts (stride 1 or a stride dividing H and W, padding (k-1)/2,
odd kernels, fp32 or bf16 on a CUDA device); anything else raises GfError from the
library call.  An input in torch's channels_last memory format takes the library's
channels-last (NHWC) kernels where they apply (r >= 2, stride 1, channel counts in multiples
of 8, dense or depthwise) and is made contiguous otherwise.
"""
from __future__ import annotations

import torch

from . import binding as B


class _FilteredConv2dFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, weight, r: int, groups: int, stride: int = 1):
        if not (x.is_cuda and weight.is_cuda):
            raise RuntimeError("filtered_conv2d needs CUDA tensors: there is no CPU path")
        ctx.need_gx = x.requires_grad          # before any copy: a copy made in here tracks no gradient
        ctx.need_gw = weight.requires_grad
        weight = weight.contiguous()
        C_out, _, KH, KW = weight.shape
        N, C_in, H, W = x.shape
        desc, fmt = None, torch.contiguous_format
        if not x.is_contiguous() and x.is_contiguous(memory_format=torch.channels_last):
            desc = B.make_desc(N, C_in, C_out, H, W, KH, KW, r=r, groups=groups, stride=stride, dtype=x.dtype,
                               layout=B.GF_NHWC)
            try:
                B.gf_backward_workspace_bytes(desc)
                fmt = torch.channels_last
            except B.GfError as e:
                if e.status != B.GF_ERR_UNSUPPORTED:
                    raise
                desc = None
        if desc is None:
            x = x.contiguous()
            desc = B.make_desc(N, C_in, C_out, H, W, KH, KW, r=r, groups=groups, stride=stride, dtype=x.dtype)
        stash = torch.empty(B.gf_stash_dims(desc), dtype=x.dtype, device=x.device, memory_format=fmt)
        stream = torch.cuda.current_stream(x.device)
        with torch.cuda.device(x.device):
            B.gf_stash_forward(desc, x, stash, stream)
        y = torch.nn.functional.conv2d(x, weight, None, stride, ((KH - 1) // 2, (KW - 1) // 2), 1, groups)
        ctx.desc = desc
        ctx.fmt = fmt
        ctx.save_for_backward(stash, weight)        # x itself is not kept
        return y

    @staticmethod
    def backward(ctx, g_y):
        stash, weight = ctx.saved_tensors
        desc = ctx.desc
        g_y = g_y.contiguous(memory_format=ctx.fmt)
        dev = g_y.device
        g_W = torch.empty(weight.shape, dtype=torch.float32, device=dev) if ctx.need_gw else None
        g_X = (torch.empty((desc.N, desc.C_in, desc.H, desc.W), dtype=g_y.dtype, device=dev, memory_format=ctx.fmt)
               if ctx.need_gx else None)
        ws = torch.empty(B.gf_backward_workspace_bytes(desc), dtype=torch.uint8, device=dev)
        stream = torch.cuda.current_stream(dev)
        with torch.cuda.device(dev):
            B.gf_backward(desc, g_y, stash, weight, g_W, g_X, ws, None, stream)
        if g_W is not None and g_W.dtype != weight.dtype:
            g_W = g_W.to(weight.dtype)
        return g_X, g_W, None, None, None


def filtered_conv2d(x: torch.Tensor, weight: torch.Tensor, r: int = 2, groups: int = 1, stride: int = 1) -> torch.Tensor:
    """conv2d(x, weight) with padding (k-1)/2 and the given stride whose gradients are the
    filtered ones with patch size r (r = 1: the exact gradients).  The bias, if any, is added
    by the caller (its gradient is not affected by the method)."""
    return _FilteredConv2dFn.apply(x, weight, int(r), int(groups), int(stride))


class FilteredConv2d(torch.nn.Module):
    """Drop-in for nn.Conv2d(..., padding=k//2) in the layers that are fine-tuned."""

    def __init__(self, in_channels: int, out_channels: int, kernel_size: int, r: int = 2, groups: int = 1,
                 bias: bool = True, device=None, dtype=None, stride: int = 1):
        super().__init__()
        self.r, self.groups, self.stride = r, groups, stride
        self.weight = torch.nn.Parameter(torch.empty(out_channels, in_channels // groups, kernel_size, kernel_size,
                                                     device=device, dtype=dtype))
        torch.nn.init.kaiming_normal_(self.weight)
        self.bias = torch.nn.Parameter(torch.zeros(out_channels, device=device, dtype=dtype)) if bias else None

    def forward(self, x):
        y = filtered_conv2d(x, self.weight, self.r, self.groups, self.stride)
        return y if self.bias is None else y + self.bias.view(1, -1, 1, 1)
