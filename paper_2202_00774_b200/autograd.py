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


class _SDGPConv2dReLUFn(torch.autograd.Function):
    """``relu(conv2d(x, weight))``, optionally followed by 2 x 2 max pooling. The backward pass forms the
    convolution's dL/dO from the gradient above the ReLU (or above the pooling) with the library's producer, which
    writes the unpruned dL/dO - the weight gradient's operand (Section 3.1) - and its compressed pruned copy in one
    pass; the sparse contraction then gives the input gradient (Section 2.1, Fig. 2)."""

    @staticmethod
    def forward(ctx, x, weight, stride, padding, pool, n, m, scheme, seed):
        act = torch.relu(torch.nn.functional.conv2d(x, weight, None, stride, padding))
        act = act.contiguous(memory_format=torch.channels_last)
        ctx.save_for_backward(x, weight, act)
        ctx.cfg = (stride, padding, pool, n, m, scheme, seed)
        return torch.nn.functional.max_pool2d(act, 2) if pool else act

    @staticmethod
    def backward(ctx, grad_out):
        x, weight, act = ctx.saved_tensors
        stride, padding, pool, n, m, scheme, seed = ctx.cfg
        dt = _dtype_code(grad_out)
        B, Cin, H, Wd = x.shape
        Cout, _, R, S = weight.shape
        P, Q = act.shape[2], act.shape[3]
        dY = grad_out.contiguous(memory_format=torch.channels_last).permute(0, 2, 3, 1)   # NHWC views
        a = act.permute(0, 2, 3, 1)
        dO = torch.empty((B, P, Q, Cout), dtype=dY.dtype, device=dY.device)
        compressed = n <= 2 and Cout % 128 == 0 and ctx.needs_input_grad[0]
        vals = torch.empty((B, P, Q, Cout // 2), dtype=dY.dtype, device=dY.device) if compressed else None
        meta = torch.empty((B, P, Q, Cout // 16), dtype=torch.int16, device=dY.device) if compressed else None
        pn, pm = (n, m) if compressed else (4, 4)   # n == m: nothing is pruned, the producer only writes dL/dO
        if pool:
            _b.sdgp_maxpool_relu_backward_prune(dY, a, pn, pm, scheme, seed, dt, grad=dO, values=vals, meta=meta)
        else:
            _b.sdgp_relu_backward_prune(dY, a, pn, pm, scheme, seed, dt, grad=dO, values=vals, meta=meta)
        grad_x = grad_w = None
        if ctx.needs_input_grad[0]:
            W = weight.contiguous(memory_format=torch.channels_last).permute(0, 2, 3, 1)   # [Cout,R,S,Cin]
            dD = torch.empty((B, H, Wd, Cin), dtype=dY.dtype, device=dY.device)
            if compressed:
                _b.sdgp_spmm_conv2d_typed(vals, meta, W, dD, stride, padding, dt)
            else:   # no compressed form to hand over: prune dL/dO in a pass of its own
                ws = torch.empty(max(16, _b.sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, stride, padding,
                                                                       _b.FLAG_TWO_PASS if n <= 2 else _b.FLAG_MASKED)),
                                 dtype=torch.uint8, device=dY.device)
                _b.sdgp_dgrad_conv2d_typed(dO, W, dD, stride, padding, n, m, scheme, seed, dt, workspace=ws,
                                           flags=_b.FLAG_TWO_PASS if n <= 2 else _b.FLAG_MASKED)
            grad_x = dD.permute(0, 3, 1, 2)
        if ctx.needs_input_grad[1]:
            grad_w = torch.nn.grad.conv2d_weight(x, weight.shape, dO.permute(0, 3, 1, 2), stride, padding)   # unpruned dL/dO
        return grad_x, grad_w, None, None, None, None, None, None, None


def sdgp_conv2d_relu(x, weight, stride=1, padding=0, pool=False, n=2, m=4, scheme=_b.MAGNITUDE, seed=0):
    """``relu(conv2d(x, weight))`` - with ``pool=True`` followed by ``max_pool2d(., 2)`` - whose backward pass
    forms and prunes the convolution's dL/dO in one pass over the incoming gradient (ReLU backward, pooling
    backward and Algorithm 1 together) and computes the input gradient from the pruned copy. Same tensor
    requirements as ``sdgp_conv2d``; with ``pool=True`` the convolution's output height and width must be even."""
    return _SDGPConv2dReLUFn.apply(x, weight, stride, padding, pool, n, m, scheme, seed)
