"""Pins for the oracle's data-gradient contraction (Section 2.1, Fig. 2 and Fig. 3)."""
import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs

torch = pytest.importorskip("torch")


def f64(b):
    return inputs.bf16_bits_to_f32(b).astype(np.float64)


def rel_fro(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def library_conv_dgrad(dOp_bits, W_bits, H, Wd, stride, pad):
    """fp64 library routine: gradient of conv2d w.r.t. its input."""
    g = torch.from_numpy(f64(dOp_bits)).permute(0, 3, 1, 2).contiguous()           # NCHW
    w = torch.from_numpy(f64(W_bits)).permute(0, 3, 1, 2).contiguous()             # [Cout,Cin,R,S]
    B, Cin = g.shape[0], w.shape[1]
    dx = torch.nn.grad.conv2d_input((B, Cin, H, Wd), w, g, stride=stride, padding=pad)
    return dx.permute(0, 2, 3, 1).contiguous().numpy()


def test_linear_equals_library_matmul():
    dO, W = inputs.fc_tensors(37, 96, 50, seed=3)
    assert rel_fro(oracle.dgrad_linear(dO, W), f64(dO) @ f64(W)) < 1e-14


def test_linear_is_not_transposed():
    # one-hot rows pick out rows of W: dD[r, :] = W[k, :] when dOp[r, :] = e_k
    K, N = 16, 8
    W = inputs.normal_bf16((K, N), 1.0, seed=1)
    eye = inputs.f32_to_bf16_bits(np.eye(K, dtype=np.float32))
    assert np.array_equal(oracle.dgrad_linear(eye, W), f64(W))


def test_linear_row_subset():
    dO, W = inputs.fc_tensors(64, 32, 24, seed=5)
    full = oracle.dgrad_linear(dO, W)
    idx = np.array([5, 0, 63, 17])
    assert np.array_equal(oracle.dgrad_linear(dO, W, row_index=idx), full[idx])


def test_pruned_linear_equals_matmul_of_pruned_copy():
    dO, W = inputs.fc_tensors(32, 64, 16, seed=6)
    p = oracle.prune(dO, 2, 4, oracle.MAGNITUDE, want=("dense",))["dense"]
    assert rel_fro(oracle.dgrad_linear(p, W), f64(p) @ f64(W)) < 1e-14
    # N == M prunes nothing: the dense path
    d = oracle.prune(dO, 4, 4, oracle.MAGNITUDE, want=("dense",))["dense"]
    assert np.array_equal(d, dO)


@pytest.mark.parametrize("B,H,Wd,Cin,Cout,R,S,stride,pad", [
    (2, 6, 5, 3, 4, 3, 3, 1, 1),
    (1, 8, 8, 5, 2, 1, 1, 1, 0),
    (2, 7, 9, 4, 6, 3, 3, 2, 1),
    (1, 8, 8, 3, 3, 1, 1, 2, 0),
    (1, 9, 7, 2, 3, 5, 3, 1, 2),
    (2, 5, 5, 2, 2, 3, 3, 1, 0),
])
def test_conv_equals_library_transposed_convolution(B, H, Wd, Cin, Cout, R, S, stride, pad):
    P, Q = (H + 2 * pad - R) // stride + 1, (Wd + 2 * pad - S) // stride + 1
    dO = inputs.relu_masked_laplace_bf16((B, P, Q, Cout), seed=B + H)
    W = inputs.normal_bf16((Cout, R, S, Cin), 0.3, seed=Cin)
    got = oracle.dgrad_conv2d(dO, W, H, Wd, stride, pad)
    assert rel_fro(got, library_conv_dgrad(dO, W, H, Wd, stride, pad)) < 1e-13


def test_conv_1x1_reduces_to_linear():
    B, H, Wd, Cin, Cout = 2, 4, 3, 6, 8
    dO = inputs.normal_bf16((B, H, Wd, Cout), 1.0, seed=1)
    W = inputs.normal_bf16((Cout, 1, 1, Cin), 1.0, seed=2)
    conv = oracle.dgrad_conv2d(dO, W, H, Wd, 1, 0).reshape(-1, Cin)
    lin = oracle.dgrad_linear(dO.reshape(-1, Cout), W.reshape(Cout, Cin))
    assert np.array_equal(conv, lin)


def test_conv_one_hot_filter_is_a_shift():
    # W[co, r0, s0, ci] = [co == ci]: dD[b,h,w,:] = dOp[b, h+pad-r0, w+pad-s0, :] (zero outside)
    B, H, Wd, C, R, S, pad = 1, 5, 6, 3, 3, 3, 1
    dO = inputs.normal_bf16((B, H, Wd, C), 1.0, seed=4)
    for r0 in range(R):
        for s0 in range(S):
            Wf = np.zeros((C, R, S, C), np.float32)
            for c in range(C):
                Wf[c, r0, s0, c] = 1.0
            got = oracle.dgrad_conv2d(dO, inputs.f32_to_bf16_bits(Wf), H, Wd, 1, pad)
            want = np.zeros((B, H, Wd, C))
            src = f64(dO)
            for h in range(H):
                for w in range(Wd):
                    p, q = h + pad - r0, w + pad - s0
                    if 0 <= p < H and 0 <= q < Wd:
                        want[0, h, w] = src[0, p, q]
            assert np.array_equal(got, want)


@pytest.mark.parametrize("stride,pad,R", [(1, 1, 3), (2, 1, 3), (2, 0, 1)])
def test_conv_adjoint_identity(stride, pad, R):
    """<conv_forward(D), G> == <D, dgrad(G)> for the forward layer the gradient belongs to."""
    B, H, Wd, Cin, Cout = 2, 7, 6, 3, 4
    P, Q = (H + 2 * pad - R) // stride + 1, (Wd + 2 * pad - R) // stride + 1
    rng = np.random.default_rng(0)
    D = rng.standard_normal((B, H, Wd, Cin))
    G = inputs.normal_bf16((B, P, Q, Cout), 1.0, seed=8)
    W = inputs.normal_bf16((Cout, R, R, Cin), 0.5, seed=9)
    lhs = (oracle.conv2d_forward_f64(D, W, stride, pad) * f64(G)).sum()
    rhs = (D * oracle.dgrad_conv2d(G, W, H, Wd, stride, pad)).sum()
    assert abs(lhs - rhs) <= 1e-12 * max(abs(lhs), 1.0)


def test_conv_forward_helper_equals_library():
    B, H, Wd, Cin, Cout, R = 1, 6, 6, 2, 3, 3
    rng = np.random.default_rng(1)
    D = rng.standard_normal((B, H, Wd, Cin))
    W = inputs.normal_bf16((Cout, R, R, Cin), 0.5, seed=3)
    got = oracle.conv2d_forward_f64(D, W, 1, 1)
    ref = torch.nn.functional.conv2d(torch.from_numpy(D).permute(0, 3, 1, 2),
                                     torch.from_numpy(f64(W)).permute(0, 3, 1, 2), stride=1, padding=1)
    assert rel_fro(got, ref.permute(0, 2, 3, 1).numpy()) < 1e-14


def test_conv_linearity_in_power_of_two():
    B, H, Wd, Cin, Cout = 1, 4, 4, 2, 4
    dO = inputs.normal_bf16((B, H, Wd, Cout), 1.0, seed=1)
    W = inputs.normal_bf16((Cout, 3, 3, Cin), 1.0, seed=2)
    dO4 = inputs.f32_to_bf16_bits(inputs.bf16_bits_to_f32(dO) * 4.0)
    assert np.array_equal(oracle.dgrad_conv2d(dO4, W, H, Wd, 1, 1), 4.0 * oracle.dgrad_conv2d(dO, W, H, Wd, 1, 1))


def test_conv_pixel_subset():
    B, H, Wd, Cin, Cout = 2, 5, 4, 3, 4
    dO = inputs.normal_bf16((B, H, Wd, Cout), 1.0, seed=1)
    W = inputs.normal_bf16((Cout, 3, 3, Cin), 1.0, seed=2)
    full = oracle.dgrad_conv2d(dO, W, H, Wd, 1, 1).reshape(-1, Cin)
    idx = np.array([0, 39, 17, 4])
    assert np.array_equal(oracle.dgrad_conv2d(dO, W, H, Wd, 1, 1, pixel_index=idx), full[idx])
