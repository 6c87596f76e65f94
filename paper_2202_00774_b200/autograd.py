"""``torch.autograd`` front end: layers whose backward pass prunes the incoming output gradient
and computes the input gradient with the SDGP kernels (Algorithm 1; Section 3.1: "SDGP only
changes the data gradient; the weight gradient uses the unpruned dL/dO").

Only the data gradient runs in this library. The forward pass and the weight gradient are the
framework's own operators, untouched, which is the integration the paper describes (Section 1:
a drop-in change of the backward pass). Tensors are bf16 or fp16 CUDA tensors; convolutions use
the channels-last memory format (its physical layout is the NHWC / [Cout,R,S,Cin] layout of the
C ABI, so nothing is copied or transposed).
"""
from __future__ import annotations

import torch

from . import binding as _b


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return _b.BF16
    if t.dtype == torch.float16:
        return _b.FP16
    raise TypeError("SDGP layers take bfloat16 or float16 tensors, got %s" % t.dtype)


class _SDGPLinearFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, weight, n, m, scheme, seed):
        ctx.save_for_backward(x, weight)
        ctx.cfg = (n, m, scheme, seed)
        return x @ weight.t()

    @staticmethod
    def backward(ctx, grad_out):
        x, weight = ctx.saved_tensors
        n, m, scheme, seed = ctx.cfg
        dO = grad_out.reshape(-1, weight.shape[0]).contiguous()
        grad_x = grad_w = None
        if ctx.needs_input_grad[0]:
            rows, K = dO.shape
            N = weight.shape[1]
            dD = torch.empty((rows, N), dtype=dO.dtype, device=dO.device)
            ws = torch.empty(max(16, _b.sdgp_workspace_size_linear(rows, K, N)), dtype=torch.uint8, device=dO.device)
            # weight is [out_features, in_features] = [K, N]: the layout sdgp_dgrad_linear wants
            _b.sdgp_dgrad_linear_typed(dO, weight.contiguous(), dD, n, m, scheme, seed, _dtype_code(dO), workspace=ws)
            grad_x = dD.reshape(x.shape)
        if ctx.needs_input_grad[1]:
            grad_w = dO.t() @ x.reshape(-1, x.shape[-1])   # unpruned dL/dO (Section 3.1)
        return grad_x, grad_w, None, None, None, None


def sdgp_linear(x, weight, n=2, m=4, scheme=_b.MAGNITUDE, seed=0):
    """``x @ weight.T`` whose input gradient is ``prune(dL/dO) @ weight`` (N:M along out_features).
    in_features and out_features must be multiples of 64."""
    return _SDGPLinearFn.apply(x, weight, n, m, scheme, seed)


class _SDGPConv2dFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, weight, stride, padding, n, m, scheme, seed):
        ctx.save_for_backward(x, weight)
        ctx.cfg = (stride, padding, n, m, scheme, seed)
        return torch.nn.functional.conv2d(x, weight, None, stride, padding)

    @staticmethod
    def backward(ctx, grad_out):
        x, weight = ctx.saved_tensors
        stride, padding, n, m, scheme, seed = ctx.cfg
        grad_x = grad_w = None
        if ctx.needs_input_grad[0]:
            # channels-last NCHW tensors are NHWC in memory: permuted views, no copies when the
            # tensors already have that format
            dO = grad_out.contiguous(memory_format=torch.channels_last).permute(0, 2, 3, 1)
            W = weight.contiguous(memory_format=torch.channels_last).permute(0, 2, 3, 1)   # [Cout,R,S,Cin]
            B, Cin, H, Wd = x.shape
            Cout, _, R, S = weight.shape
            dD = torch.empty((B, H, Wd, Cin), dtype=dO.dtype, device=dO.device)
            ws = torch.empty(max(16, _b.sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, stride, padding)),
                             dtype=torch.uint8, device=dO.device)
            _b.sdgp_dgrad_conv2d_typed(dO, W, dD, stride, padding, n, m, scheme, seed, _dtype_code(dO), workspace=ws)
            grad_x = dD.permute(0, 3, 1, 2)   # NCHW view of channels-last storage
        if ctx.needs_input_grad[1]:
            grad_w = torch.nn.grad.conv2d_weight(x, weight.shape, grad_out, stride, padding)   # unpruned dL/dO
        return grad_x, grad_w, None, None, None, None, None, None


def sdgp_conv2d(x, weight, stride=1, padding=0, n=2, m=4, scheme=_b.MAGNITUDE, seed=0):
    """``conv2d(x, weight)`` (NCHW tensors, channels-last storage recommended, no bias, stride 1 or 2,
    one padding value for both axes) whose input gradient is computed from dL/dO pruned N:M along
    the output channels. Channel counts must be multiples of 64."""
    return _SDGPConv2dFn.apply(x, weight, stride, padding, n, m, scheme, seed)
