"""Python binding of the SDGP C ABI (``include/sdgp.h``): argument marshalling only.

Tensors are torch CUDA tensors (device memory and streams come from torch); every
computation happens inside ``libsdgp.so``. There is no fallback: a missing library or a
non-OK status raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

RANDOM, MAGNITUDE, RESCALED_MAGNITUDE = 0, 1, 2
FLAG_TWO_PASS, FLAG_FUSED, FLAG_DENSE, FLAG_MASKED, FLAG_CHANNEL = 0, 1, 2, 3, 4

BF16, FP16 = 0, 1   # sdgp_dtype
EXPORTS = ["sdgp_prune", "sdgp_dgrad_linear", "sdgp_dgrad_conv2d", "sdgp_spmm_linear", "sdgp_spmm_conv2d",
           "sdgp_prune_typed", "sdgp_dgrad_linear_typed", "sdgp_dgrad_conv2d_typed", "sdgp_spmm_linear_typed",
           "sdgp_spmm_conv2d_typed", "sdgp_channel_scales", "sdgp_relu_backward_prune", "sdgp_residual_relu_backward_prune", "sdgp_maxpool_relu_backward_prune", "sdgp_dgrad_linear_static", "sdgp_selftest_bounded_wait",
           "sdgp_workspace_size_linear", "sdgp_workspace_size_conv2d", "sdgp_workspace_size_conv2d_grouped",
           "sdgp_dgrad_conv2d_grouped", "sdgp_last_device_error",
           "sdgp_status_string"]

_lib = None


class SdgpError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__("%s failed: %s (status %d)" % (what, status_string(status), status))
        self.status = status


def lib() -> ctypes.CDLL:
    """Loads (building first if the sources are newer) the C-ABI library."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if _build.needs_build():
            path = _build.build()
        if not os.path.exists(path):
            raise RuntimeError("libsdgp.so is missing; run paper_2202_00774_b200/build.py")
        L = ctypes.CDLL(path)
        i64, u64, i32, u32, vp, sz = (ctypes.c_int64, ctypes.c_uint64, ctypes.c_int, ctypes.c_uint32,
                                      ctypes.c_void_p, ctypes.c_size_t)
        L.sdgp_prune.argtypes = [vp, i64, i64, i32, i32, i32, u64, vp, vp, vp, vp, vp]
        L.sdgp_prune.restype = i32
        L.sdgp_dgrad_linear.argtypes = [vp, vp, vp, i64, i64, i64, i32, i32, i32, u64, vp, sz, u32, vp]
        L.sdgp_dgrad_linear.restype = i32
        L.sdgp_dgrad_conv2d.argtypes = [vp, vp, vp] + [i32] * 9 + [i32, i32, i32, u64, vp, sz, u32, vp]
        L.sdgp_dgrad_conv2d.restype = i32
        L.sdgp_dgrad_linear_static.argtypes = [vp, vp, vp, i64, i64, i64, i32, i32, i32, u64, vp]
        L.sdgp_dgrad_linear_static.restype = i32
        L.sdgp_spmm_linear.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp]
        L.sdgp_spmm_linear.restype = i32
        L.sdgp_spmm_conv2d.argtypes = [vp, vp, vp, vp] + [i32] * 9 + [vp]
        L.sdgp_spmm_conv2d.restype = i32
        L.sdgp_prune_typed.argtypes = [vp, i64, i64, i32, i32, i32, u64, i32, vp, vp, vp, vp, vp]
        L.sdgp_prune_typed.restype = i32
        L.sdgp_dgrad_linear_typed.argtypes = [vp, vp, vp, i64, i64, i64, i32, i32, i32, u64, i32, vp, sz, u32, vp]
        L.sdgp_dgrad_linear_typed.restype = i32
        L.sdgp_dgrad_conv2d_typed.argtypes = [vp, vp, vp] + [i32] * 9 + [i32, i32, i32, u64, i32, vp, sz, u32, vp]
        L.sdgp_dgrad_conv2d_typed.restype = i32
        L.sdgp_spmm_linear_typed.argtypes = [vp, vp, vp, vp, i64, i64, i64, i32, vp]
        L.sdgp_spmm_linear_typed.restype = i32
        L.sdgp_spmm_conv2d_typed.argtypes = [vp, vp, vp, vp] + [i32] * 9 + [i32, vp]
        L.sdgp_spmm_conv2d_typed.restype = i32
        L.sdgp_channel_scales.argtypes = [vp, i64, i64, i32, i32, i32, vp, vp]
        L.sdgp_relu_backward_prune.argtypes = [vp, vp, i64, i64, i32, i32, i32, u64, i32, vp, vp, vp, vp, vp, vp]
        L.sdgp_relu_backward_prune.restype = i32
        L.sdgp_residual_relu_backward_prune.argtypes = [vp, vp, vp, i64, i64, i32, i32, i32, u64, i32, vp, vp, vp, vp, vp, vp]
        L.sdgp_residual_relu_backward_prune.restype = i32
        L.sdgp_maxpool_relu_backward_prune.argtypes = [vp, vp, vp, i32, i32, i32, i64, i32, i32, i32, u64, i32, vp, vp, vp, vp, vp, vp]
        L.sdgp_maxpool_relu_backward_prune.restype = i32
        L.sdgp_channel_scales.restype = i32
        L.sdgp_workspace_size_linear.argtypes = [i64, i64, i64, u32]
        L.sdgp_workspace_size_linear.restype = sz
        L.sdgp_workspace_size_conv2d.argtypes = [i32] * 9 + [u32]
        L.sdgp_workspace_size_conv2d.restype = sz
        L.sdgp_workspace_size_conv2d_grouped.argtypes = [i32] * 10 + [u32]
        L.sdgp_workspace_size_conv2d_grouped.restype = sz
        L.sdgp_dgrad_conv2d_grouped.argtypes = [vp, vp, vp] + [i32] * 10 + [i32, i32, i32, u64, i32, vp, sz, u32, vp]
        L.sdgp_dgrad_conv2d_grouped.restype = i32
        L.sdgp_last_device_error.argtypes = []
        L.sdgp_last_device_error.restype = i32
        L.sdgp_selftest_bounded_wait.argtypes = [vp]
        L.sdgp_selftest_bounded_wait.restype = i32
        L.sdgp_status_string.argtypes = [i32]
        L.sdgp_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().sdgp_status_string(int(status)).decode()


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, what: str):
    if status != 0:
        raise SdgpError(status, what)


def _dev(t, name):
    if t is not None and (not t.is_cuda or not t.is_contiguous()):
        raise ValueError("%s must be a contiguous CUDA tensor" % name)


def sdgp_prune(dO, n, m, scheme, seed=0, dense=None, values=None, meta=None, mask=None):
    """``sdgp_prune`` of sdgp.h. ``dO`` is a 2-byte-element tensor whose last dimension is K;
    outputs are caller-allocated tensors (or None)."""
    for t, name in ((dO, "dO"), (dense, "dense"), (values, "values"), (meta, "meta"), (mask, "mask")):
        _dev(t, name)
    K = dO.shape[-1] if dO.dim() else 0
    rows = dO.numel() // K if K else 0
    _check(lib().sdgp_prune(_ptr(dO), rows, K, n, m, scheme, seed, _ptr(dense), _ptr(values), _ptr(meta),
                            _ptr(mask), _stream()), "sdgp_prune")


def sdgp_workspace_size_linear(rows, K, N, flags=FLAG_TWO_PASS) -> int:
    return int(lib().sdgp_workspace_size_linear(rows, K, N, flags))


def sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, stride, pad, flags=FLAG_TWO_PASS) -> int:
    return int(lib().sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, stride, pad, flags))


def sdgp_dgrad_linear(dO, W, dD, n, m, scheme, seed=0, workspace=None, flags=FLAG_TWO_PASS):
    """``sdgp_dgrad_linear``: dO [rows,K], W [K,N], dD [rows,N] (bf16 or 2-byte views)."""
    for t, name in ((dO, "dO"), (W, "W"), (dD, "dD"), (workspace, "workspace")):
        _dev(t, name)
    rows, K = dO.shape
    N = W.shape[1]
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().sdgp_dgrad_linear(_ptr(dO), _ptr(W), _ptr(dD), rows, K, N, n, m, scheme, seed,
                                   _ptr(workspace), ws_bytes, flags, _stream()), "sdgp_dgrad_linear")


def sdgp_dgrad_linear_static(dO, W, dD, n, m, scheme, seed=0):
    """``sdgp_dgrad_linear_static``: like :func:`sdgp_dgrad_linear` in two-pass mode, but the
    scratch is the library's own fixed device array - for callers that cannot allocate a
    workspace. rows*K is limited to 8Mi elements; calls must not overlap on the GPU."""
    for t, name in ((dO, "dO"), (W, "W"), (dD, "dD")):
        _dev(t, name)
    rows, K = dO.shape
    N = W.shape[1]
    _check(lib().sdgp_dgrad_linear_static(_ptr(dO), _ptr(W), _ptr(dD), rows, K, N, n, m, scheme, seed,
                                          _stream()), "sdgp_dgrad_linear_static")


def sdgp_dgrad_conv2d(dO, W, dD, stride, pad, n, m, scheme, seed=0, workspace=None, flags=FLAG_TWO_PASS):
    """``sdgp_dgrad_conv2d``: dO NHWC [B,P,Q,Cout], W [Cout,R,S,Cin], dD NHWC [B,H,Wd,Cin]."""
    for t, name in ((dO, "dO"), (W, "W"), (dD, "dD"), (workspace, "workspace")):
        _dev(t, name)
    B, H, Wd, Cin = dD.shape
    Cout, R, S, _ = W.shape
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().sdgp_dgrad_conv2d(_ptr(dO), _ptr(W), _ptr(dD), B, H, Wd, Cin, Cout, R, S, stride, pad, n, m,
                                   scheme, seed, _ptr(workspace), ws_bytes, flags, _stream()),
           "sdgp_dgrad_conv2d")


def sdgp_spmm_linear(values, meta, W, dD):
    for t, name in ((values, "values"), (meta, "meta"), (W, "W"), (dD, "dD")):
        _dev(t, name)
    rows, N = dD.shape
    K = W.shape[0]
    _check(lib().sdgp_spmm_linear(_ptr(values), _ptr(meta), _ptr(W), _ptr(dD), rows, K, N, _stream()),
           "sdgp_spmm_linear")


def sdgp_spmm_conv2d(values, meta, W, dD, stride, pad):
    for t, name in ((values, "values"), (meta, "meta"), (W, "W"), (dD, "dD")):
        _dev(t, name)
    B, H, Wd, Cin = dD.shape
    Cout, R, S, _ = W.shape
    _check(lib().sdgp_spmm_conv2d(_ptr(values), _ptr(meta), _ptr(W), _ptr(dD), B, H, Wd, Cin, Cout, R, S,
                                  stride, pad, _stream()), "sdgp_spmm_conv2d")


# ---- the same operations on tensors of an explicit element type (sdgp_dtype: BF16 or FP16) ----


def sdgp_prune_typed(dO, n, m, scheme, seed, dtype, dense=None, values=None, meta=None, mask=None):
    """``sdgp_prune_typed``: :func:`sdgp_prune` for 2-byte elements of type ``dtype``."""
    for t, name in ((dO, "dO"), (dense, "dense"), (values, "values"), (meta, "meta"), (mask, "mask")):
        _dev(t, name)
    K = dO.shape[-1] if dO.dim() else 0
    rows = dO.numel() // K if K else 0
    _check(lib().sdgp_prune_typed(_ptr(dO), rows, K, n, m, scheme, seed, dtype, _ptr(dense), _ptr(values),
                                  _ptr(meta), _ptr(mask), _stream()), "sdgp_prune_typed")


def sdgp_relu_backward_prune(dY, act, n, m, scheme, seed=0, dtype=BF16, grad=None, dense=None, values=None, meta=None,
                             mask=None):
    """``sdgp_relu_backward_prune``: dL/dO = dY where ``act`` > 0, pruned in the same pass. ``dY`` and ``act`` are
    2-byte-element tensors of the same shape whose last dimension is K; outputs are caller-allocated (or None)."""
    for t, name in ((dY, "dY"), (act, "act"), (grad, "grad"), (dense, "dense"), (values, "values"), (meta, "meta"),
                    (mask, "mask")):
        _dev(t, name)
    if dY.shape != act.shape:
        raise ValueError("dY and act must have the same shape")
    K = dY.shape[-1] if dY.dim() else 0
    rows = dY.numel() // K if K else 0
    _check(lib().sdgp_relu_backward_prune(_ptr(dY), _ptr(act), rows, K, n, m, scheme, seed, dtype, _ptr(grad), _ptr(dense),
                                          _ptr(values), _ptr(meta), _ptr(mask), _stream()), "sdgp_relu_backward_prune")


def sdgp_residual_relu_backward_prune(dY, dSkip, act, n, m, scheme, seed=0, dtype=BF16, grad=None, dense=None, values=None,
                                      meta=None, mask=None):
    """``sdgp_residual_relu_backward_prune``: dL/dO = dY + dSkip (rounded to the 16-bit type) where ``act`` > 0, pruned in
    the same pass. The three inputs are 2-byte-element tensors of the same shape whose last dimension is K."""
    for t, name in ((dY, "dY"), (dSkip, "dSkip"), (act, "act"), (grad, "grad"), (dense, "dense"), (values, "values"),
                    (meta, "meta"), (mask, "mask")):
        _dev(t, name)
    if dY.shape != act.shape or (dSkip is not None and dY.shape != dSkip.shape):   # (a missing dSkip is the library's to reject)
        raise ValueError("dY, dSkip and act must have the same shape")
    K = dY.shape[-1] if dY.dim() else 0
    rows = dY.numel() // K if K else 0
    _check(lib().sdgp_residual_relu_backward_prune(_ptr(dY), _ptr(dSkip), _ptr(act), rows, K, n, m, scheme, seed, dtype,
                                                   _ptr(grad), _ptr(dense), _ptr(values), _ptr(meta), _ptr(mask), _stream()),
           "sdgp_residual_relu_backward_prune")


def sdgp_maxpool_relu_backward_prune(dYp, act, n, m, scheme, seed=0, dtype=BF16, grad=None, dense=None, values=None, meta=None,
                                     mask=None, skip=None):
    """``sdgp_maxpool_relu_backward_prune``: ``dYp`` [B, H/2, W/2, K] is the gradient above a 2 x 2 max pooling, ``act``
    [B, H, W, K] the activation of the ReLU below it; dL/dO [B, H, W, K] is formed and pruned in one pass. ``skip``
    (optional, the shape of ``dYp``) is a second gradient added to ``dYp`` first."""
    for t, name in ((dYp, "dYp"), (act, "act"), (grad, "grad"), (dense, "dense"), (values, "values"), (meta, "meta"),
                    (mask, "mask"), (skip, "skip")):
        _dev(t, name)
    if skip is not None and skip.shape != dYp.shape:
        raise ValueError("skip must have the shape of dYp")
    if act.dim() != 4 or dYp.dim() != 4:
        raise ValueError("dYp and act must be NHWC tensors")
    B, H, W, K = act.shape
    if tuple(dYp.shape) != (B, H // 2, W // 2, K):
        raise ValueError("dYp must be [B, H/2, W/2, K]")
    _check(lib().sdgp_maxpool_relu_backward_prune(_ptr(dYp), _ptr(skip), _ptr(act), B, H, W, K, n, m, scheme, seed, dtype, _ptr(grad),
                                                  _ptr(dense), _ptr(values), _ptr(meta), _ptr(mask), _stream()),
           "sdgp_maxpool_relu_backward_prune")


def sdgp_dgrad_linear_typed(dO, W, dD, n, m, scheme, seed, dtype, workspace=None, flags=FLAG_TWO_PASS):
    for t, name in ((dO, "dO"), (W, "W"), (dD, "dD"), (workspace, "workspace")):
        _dev(t, name)
    rows, K = dO.shape
    N = W.shape[1]
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().sdgp_dgrad_linear_typed(_ptr(dO), _ptr(W), _ptr(dD), rows, K, N, n, m, scheme, seed, dtype,
                                         _ptr(workspace), ws_bytes, flags, _stream()), "sdgp_dgrad_linear_typed")


def sdgp_dgrad_conv2d_typed(dO, W, dD, stride, pad, n, m, scheme, seed, dtype, workspace=None, flags=FLAG_TWO_PASS):
    for t, name in ((dO, "dO"), (W, "W"), (dD, "dD"), (workspace, "workspace")):
        _dev(t, name)
    B, H, Wd, Cin = dD.shape
    Cout, R, S, _ = W.shape
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().sdgp_dgrad_conv2d_typed(_ptr(dO), _ptr(W), _ptr(dD), B, H, Wd, Cin, Cout, R, S, stride, pad, n, m,
                                         scheme, seed, dtype, _ptr(workspace), ws_bytes, flags, _stream()),
           "sdgp_dgrad_conv2d_typed")


def sdgp_workspace_size_conv2d_grouped(B, H, Wd, Cin, Cout, R, S, stride, pad, groups, flags=FLAG_TWO_PASS) -> int:
    return int(lib().sdgp_workspace_size_conv2d_grouped(B, H, Wd, Cin, Cout, R, S, stride, pad, groups, flags))


def sdgp_dgrad_conv2d_grouped(dO, W, dD, stride, pad, groups, n, m, scheme, seed=0, dtype=BF16, workspace=None,
                              flags=FLAG_TWO_PASS):
    """``sdgp_dgrad_conv2d_grouped``: dO NHWC [B,P,Q,Cout], W [Cout,R,S,Cin/groups], dD NHWC [B,H,W,Cin]."""
    for t, name in ((dO, "dO"), (W, "W"), (dD, "dD"), (workspace, "workspace")):
        _dev(t, name)
    B, H, Wd, Cin = dD.shape
    Cout, R, S, _ = W.shape
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().sdgp_dgrad_conv2d_grouped(_ptr(dO), _ptr(W), _ptr(dD), B, H, Wd, Cin, Cout, R, S, stride, pad, groups,
                                           n, m, scheme, seed, dtype, _ptr(workspace), ws_bytes, flags, _stream()),
           "sdgp_dgrad_conv2d_grouped")


def sdgp_spmm_linear_typed(values, meta, W, dD, dtype):
    for t, name in ((values, "values"), (meta, "meta"), (W, "W"), (dD, "dD")):
        _dev(t, name)
    rows, N = dD.shape
    K = W.shape[0]
    _check(lib().sdgp_spmm_linear_typed(_ptr(values), _ptr(meta), _ptr(W), _ptr(dD), rows, K, N, dtype, _stream()),
           "sdgp_spmm_linear_typed")


def sdgp_spmm_conv2d_typed(values, meta, W, dD, stride, pad, dtype):
    for t, name in ((values, "values"), (meta, "meta"), (W, "W"), (dD, "dD")):
        _dev(t, name)
    B, H, Wd, Cin = dD.shape
    Cout, R, S, _ = W.shape
    _check(lib().sdgp_spmm_conv2d_typed(_ptr(values), _ptr(meta), _ptr(W), _ptr(dD), B, H, Wd, Cin, Cout, R, S,
                                        stride, pad, dtype, _stream()), "sdgp_spmm_conv2d_typed")


def sdgp_channel_scales(dO, n, m, dtype, out):
    """``sdgp_channel_scales``: ``out`` is a float32 CUDA tensor of 3*K elements (factors, sums of |dO|, sums over survivors)."""
    _dev(dO, "dO")
    _dev(out, "out")
    K = dO.shape[-1]
    rows = dO.numel() // K if K else 0
    if out.numel() < 3 * K or out.element_size() != 4:
        raise ValueError("out must hold 3*K float32 values")
    _check(lib().sdgp_channel_scales(_ptr(dO), rows, K, n, m, dtype, _ptr(out), _stream()), "sdgp_channel_scales")


def sdgp_selftest_bounded_wait():
    """Enqueues the kernel whose wait must run out (see sdgp.h); check with sdgp_last_device_error()."""
    _check(lib().sdgp_selftest_bounded_wait(_stream()), "sdgp_selftest_bounded_wait")


def sdgp_last_device_error() -> int:
    return int(lib().sdgp_last_device_error())
