"""ctypes front end of the CPU oracle (``sdgp_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's
CPU-baseline leg import this; the GPU library never does, and nothing here
touches the GPU library. Arrays are numpy; bf16 tensors are ``uint16`` bit
patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sdgp_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

RANDOM, MAGNITUDE, RESCALED = 0, 1, 2
BF16, FP16 = 0, 1   # element type of the 16-bit tensors (bf16 unless a call says otherwise)

_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
             "-fno-fast-math", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i64, u64, i32, vp, dbl = (ctypes.c_int64, ctypes.c_uint64, ctypes.c_int, ctypes.c_void_p,
                                      ctypes.c_double)
            lib.oracle_prune.argtypes = [vp, i64, i64, i32, i32, i32, u64, vp, vp, vp, vp]
            lib.oracle_prune.restype = i32
            lib.oracle_prune_t.argtypes = [vp, i64, i64, i32, i32, i32, i32, u64, vp, vp, vp, vp]
            lib.oracle_prune_t.restype = i32
            lib.oracle_dgrad_linear_t.argtypes = [vp, vp, vp, i64, i64, i64, vp, i64, i32, vp]
            lib.oracle_dgrad_linear_t.restype = i32
            lib.oracle_dgrad_conv2d_t.argtypes = [vp, vp, vp] + [i32] * 9 + [vp, i64, i32, vp]
            lib.oracle_channel_scales.argtypes = [vp, i64, i64, i32, i32, i32, vp]
            lib.oracle_channel_scales.restype = i32
            lib.oracle_dgrad_conv2d_t.restype = i32
            lib.oracle_dgrad_conv2d_grouped_t.argtypes = [vp, vp, vp] + [i32] * 10 + [vp, i64, i32]
            lib.oracle_dgrad_conv2d_grouped_t.restype = i32
            lib.oracle_f32_to_f16.argtypes = [ctypes.c_float]
            lib.oracle_f32_to_f16.restype = ctypes.c_uint16
            lib.oracle_f16_to_f64.argtypes = [ctypes.c_uint16]
            lib.oracle_f16_to_f64.restype = dbl
            lib.oracle_relu_backward.argtypes = [vp, vp, i64, i32, vp]
            lib.oracle_relu_backward.restype = i32
            lib.oracle_residual_relu_backward.argtypes = [vp, vp, vp, i64, i32, vp]
            lib.oracle_residual_relu_backward.restype = i32
            lib.oracle_maxpool_relu_backward.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp]
            lib.oracle_maxpool_relu_backward.restype = i32
            lib.oracle_expand.argtypes = [vp, vp, i64, i64, vp]
            lib.oracle_expand.restype = i32
            lib.oracle_dgrad_linear.argtypes = [vp, vp, vp, i64, i64, i64, vp, i64]
            lib.oracle_dgrad_linear.restype = i32
            lib.oracle_dgrad_conv2d.argtypes = [vp, vp, vp] + [i32] * 9 + [vp, i64]
            lib.oracle_dgrad_conv2d.restype = i32
            lib.oracle_conv2d_forward_f64.argtypes = [vp, vp, vp] + [i32] * 9
            lib.oracle_conv2d_forward_f64.restype = i32
            lib.oracle_philox4x32_10.argtypes = [vp, vp, vp]
            lib.oracle_philox4x32_10.restype = None
            lib.oracle_random_key16.argtypes = [u64, u64]
            lib.oracle_random_key16.restype = ctypes.c_uint16
            lib.oracle_f32_to_bf16.argtypes = [ctypes.c_float]
            lib.oracle_f32_to_bf16.restype = ctypes.c_uint16
            lib.oracle_bf16_to_f64.argtypes = [ctypes.c_uint16]
            lib.oracle_bf16_to_f64.restype = dbl
            lib.oracle_runtime_reduction.argtypes = [dbl, i32, i32]
            lib.oracle_runtime_reduction.restype = dbl
            _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a, shape=None):
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("bf16 tensors are passed as uint16 bit patterns")
    return a if shape is None else a.reshape(shape)


def compressible(n: int, m: int) -> bool:
    return n <= 2 and m % 4 == 0


def prune(dO, n, m, scheme, seed=0, want=("dense", "values", "meta", "mask"), dtype=BF16):
    """Algorithm 1 with the Section 3.2 pruning function ``scheme`` on a
    ``[rows, K]`` uint16 array of ``dtype`` elements. Returns a dict with the requested outputs."""
    dO = _u16(dO)
    rows, K = dO.shape
    out = {}
    if "dense" in want:
        out["dense"] = np.empty((rows, K), np.uint16)
    if "values" in want:
        out["values"] = np.empty((rows, K // 2), np.uint16)
    if "meta" in want:
        out["meta"] = np.empty((rows, K // 16), np.uint16)
    if "mask" in want:
        out["mask"] = np.empty((rows, K // 32), np.uint32)
    rc = _load().oracle_prune_t(_ptr(dO), rows, K, n, m, scheme, dtype, seed, _ptr(out.get("dense")),
                                _ptr(out.get("values")), _ptr(out.get("meta")), _ptr(out.get("mask")))
    if rc != 0:
        raise ValueError("oracle_prune rejected its arguments (rc=%d)" % rc)
    return out


def relu_backward(dY, act, dtype=BF16):
    """dL/dO below a ReLU (Section 2.1, Fig. 2): dY where the ReLU's activation ``act`` is positive, +0.0 elsewhere.
    Arrays of 16-bit patterns of the same shape."""
    dY, act = _u16(dY), _u16(act)
    if dY.shape != act.shape:
        raise ValueError("dY and act must have the same shape")
    out = np.empty(dY.shape, np.uint16)
    rc = _load().oracle_relu_backward(_ptr(dY), _ptr(act), dY.size, dtype, _ptr(out))
    if rc != 0:
        raise ValueError("oracle_relu_backward rejected its arguments")
    return out


def relu_backward_prune(dY, act, n, m, scheme, seed=0, want=("dense", "values", "meta", "mask"), dtype=BF16):
    """The producer of the pruned dL/dO: ReLU backward, then Algorithm 1 on the result. Returns the dict of
    ``prune`` plus ``"grad"``, the unpruned dL/dO that the weight gradient still needs (Section 3.1)."""
    grad = relu_backward(dY, act, dtype)
    out = prune(grad, n, m, scheme, seed, want, dtype)
    out["grad"] = grad
    return out


def residual_relu_backward(dY, dSkip, act, dtype=BF16):
    """dL/dO below the ReLU that follows a residual addition (the ResNets of Section 4): the two gradients handed down
    to the ReLU's output are added (single precision, rounded to the 16-bit type), and the sum passes where ``act`` is
    positive. Arrays of 16-bit patterns of the same shape."""
    dY, dSkip, act = _u16(dY), _u16(dSkip), _u16(act)
    if dY.shape != act.shape or dY.shape != dSkip.shape:
        raise ValueError("dY, dSkip and act must have the same shape")
    out = np.empty(dY.shape, np.uint16)
    rc = _load().oracle_residual_relu_backward(_ptr(dY), _ptr(dSkip), _ptr(act), dY.size, dtype, _ptr(out))
    if rc != 0:
        raise ValueError("oracle_residual_relu_backward rejected its arguments")
    return out


def residual_relu_backward_prune(dY, dSkip, act, n, m, scheme, seed=0, want=("dense", "values", "meta", "mask"), dtype=BF16):
    """``residual_relu_backward`` followed by Algorithm 1; ``"grad"`` is the unpruned dL/dO (Section 3.1)."""
    grad = residual_relu_backward(dY, dSkip, act, dtype)
    out = prune(grad, n, m, scheme, seed, want, dtype)
    out["grad"] = grad
    return out


def maxpool_relu_backward(dYp, act, dtype=BF16):
    """dL/dO below a ReLU that is followed by a 2 x 2 max pooling of stride 2 (ResNet-9's blocks, Section 4): ``dYp``
    [B, H/2, W/2, K] is the gradient above the pooling, ``act`` [B, H, W, K] the ReLU's activation; each pooled
    gradient goes to the first largest activation of its window if that is positive. Returns [B, H, W, K]."""
    dYp, act = _u16(dYp), _u16(act)
    B, H, W, K = act.shape
    if dYp.shape != (B, H // 2, W // 2, K) or H % 2 or W % 2:
        raise ValueError("dYp must be [B, H/2, W/2, K] for act [B, H, W, K] with even H and W")
    out = np.empty(act.shape, np.uint16)
    rc = _load().oracle_maxpool_relu_backward(_ptr(dYp), _ptr(act), B, H, W, K, dtype, _ptr(out))
    if rc != 0:
        raise ValueError("oracle_maxpool_relu_backward rejected its arguments")
    return out


def maxpool_relu_backward_prune(dYp, act, n, m, scheme, seed=0, want=("dense", "values", "meta", "mask"), dtype=BF16, skip=None):
    """``maxpool_relu_backward`` followed by Algorithm 1 along K; outputs as [B*H*W, ...]; ``"grad"`` is the unpruned
    dL/dO [B, H, W, K] (Section 3.1). ``skip``: a second gradient of the pooled shape (a residual block below the pooling),
    added to ``dYp`` first as ``residual_relu_backward`` adds (through a gate that is open everywhere)."""
    if skip is not None:
        one = np.full(np.shape(dYp), 0x3C00 if dtype == FP16 else 0x3F80, np.uint16)
        dYp = residual_relu_backward(dYp, skip, one, dtype)
    grad = maxpool_relu_backward(dYp, act, dtype)
    out = prune(grad.reshape(-1, grad.shape[-1]), n, m, scheme, seed, want, dtype)
    out["grad"] = grad
    return out


def expand(values, meta):
    values, meta = _u16(values), _u16(meta)
    rows, K = values.shape[0], values.shape[1] * 2
    dense = np.empty((rows, K), np.uint16)
    rc = _load().oracle_expand(_ptr(values), _ptr(meta), rows, K, _ptr(dense))
    if rc != 0:
        raise ValueError("oracle_expand rejected its arguments")
    return dense


def channel_scales(dO, n, m, dtype=BF16):
    """Per-channel reading of the L1 rescale: one fp64 factor per column of the ``[rows, K]`` tensor,
    sum|x| / sum|kept x| over all rows under the magnitude mask (1 where nothing of the column is kept)."""
    dO = _u16(dO)
    rows, K = dO.shape
    out = np.empty(K, np.float64)
    rc = _load().oracle_channel_scales(_ptr(dO), rows, K, n, m, dtype, _ptr(out))
    if rc != 0:
        raise ValueError("oracle_channel_scales rejected its arguments")
    return out


def _scale_arg(k_scale, K):
    if k_scale is None:
        return None
    a = np.ascontiguousarray(k_scale, dtype=np.float64)
    if a.shape != (K,):
        raise ValueError("k_scale must have one entry per output channel")
    return a


def dgrad_linear(dOp, W, row_index=None, dtype=BF16, k_scale=None):
    """dD = (dOp * k_scale) @ W in fp64 from 16-bit bit patterns; ``row_index`` evaluates a subset of rows."""
    dOp, W = _u16(dOp), _u16(W)
    rows, K = dOp.shape
    K2, N = W.shape
    if K != K2:
        raise ValueError("shape mismatch")
    idx = None if row_index is None else np.ascontiguousarray(row_index, dtype=np.int64)
    count = rows if idx is None else idx.shape[0]
    dD = np.empty((count, N), np.float64)
    ks = _scale_arg(k_scale, K)
    rc = _load().oracle_dgrad_linear_t(_ptr(dOp), _ptr(W), _ptr(dD), rows, K, N, _ptr(idx), count, dtype, _ptr(ks))
    if rc != 0:
        raise ValueError("oracle_dgrad_linear rejected its arguments")
    return dD


def dgrad_conv2d(dOp, W, H, Wd, stride=1, pad=0, pixel_index=None, dtype=BF16, k_scale=None):
    """dD (NHWC, fp64) from dOp NHWC ``[B,P,Q,Cout]`` and W ``[Cout,R,S,Cin]`` (uint16)."""
    dOp, W = _u16(dOp), _u16(W)
    B, P, Q, Cout = dOp.shape
    Cout2, R, S, Cin = W.shape
    if Cout != Cout2 or P != (H + 2 * pad - R) // stride + 1 or Q != (Wd + 2 * pad - S) // stride + 1:
        raise ValueError("shape mismatch")
    idx = None if pixel_index is None else np.ascontiguousarray(pixel_index, dtype=np.int64)
    count = B * H * Wd if idx is None else idx.shape[0]
    dD = np.empty((count, Cin), np.float64)
    ks = _scale_arg(k_scale, Cout)
    rc = _load().oracle_dgrad_conv2d_t(_ptr(dOp), _ptr(W), _ptr(dD), B, H, Wd, Cin, Cout, R, S, stride,
                                       pad, _ptr(idx), count, dtype, _ptr(ks))
    if rc != 0:
        raise ValueError("oracle_dgrad_conv2d rejected its arguments")
    return dD.reshape(B, H, Wd, Cin) if idx is None else dD


def dgrad_conv2d_grouped(dOp, W, H, Wd, groups, stride=1, pad=0, pixel_index=None, dtype=BF16):
    """dD (NHWC, fp64) of a grouped convolution: dOp NHWC ``[B,P,Q,Cout]``, W ``[Cout,R,S,Cin/groups]`` (uint16)."""
    dOp, W = _u16(dOp), _u16(W)
    B, P, Q, Cout = dOp.shape
    Cout2, R, S, cin_g = W.shape
    if Cout != Cout2 or P != (H + 2 * pad - R) // stride + 1 or Q != (Wd + 2 * pad - S) // stride + 1:
        raise ValueError("shape mismatch")
    Cin = cin_g * groups
    idx = None if pixel_index is None else np.ascontiguousarray(pixel_index, dtype=np.int64)
    count = B * H * Wd if idx is None else idx.shape[0]
    dD = np.empty((count, Cin), np.float64)
    rc = _load().oracle_dgrad_conv2d_grouped_t(_ptr(dOp), _ptr(W), _ptr(dD), B, H, Wd, Cin, Cout, R, S, stride,
                                               pad, groups, _ptr(idx), count, dtype)
    if rc != 0:
        raise ValueError("oracle_dgrad_conv2d_grouped rejected its arguments")
    return dD.reshape(B, H, Wd, Cin) if idx is None else dD


def conv2d_forward_f64(D, W, stride=1, pad=0):
    D = np.ascontiguousarray(D, dtype=np.float64)
    W = _u16(W)
    B, H, Wd, Cin = D.shape
    Cout, R, S, _ = W.shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (Wd + 2 * pad - S) // stride + 1
    O = np.empty((B, P, Q, Cout), np.float64)
    rc = _load().oracle_conv2d_forward_f64(_ptr(D), _ptr(W), _ptr(O), B, H, Wd, Cin, Cout, R, S,
                                           stride, pad)
    if rc != 0:
        raise ValueError("oracle_conv2d_forward_f64 rejected its arguments")
    return O


def philox4x32_10(ctr, key):
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    o = np.empty(4, np.uint32)
    _load().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(o))
    return o


def random_key16(seed, e):
    return int(_load().oracle_random_key16(seed, e))


def f32_to_bf16(x):
    return int(_load().oracle_f32_to_bf16(float(x)))


def bf16_to_f64(bits):
    return float(_load().oracle_bf16_to_f64(int(bits)))


def f32_to_f16(x):
    return int(_load().oracle_f32_to_f16(float(x)))


def f16_to_f64(bits):
    return float(_load().oracle_f16_to_f64(int(bits)))


def bf16_array_to_f64(a):
    """Vectorised bf16 bits -> float64 (pure bit widening)."""
    a = _u16(a)
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def runtime_reduction(share, n, m):
    """Section 4.3 closed form: share * (1 - n/m)."""
    return float(_load().oracle_runtime_reduction(share, n, m))


def omp_threads() -> int:
    return int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
