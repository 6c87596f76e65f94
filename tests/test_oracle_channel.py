"""Pins for the oracle's per-channel reading of the L1 rescale (Section 3.3 / Fig. 4 caption:
the norm is preserved per channel over batch and spatial positions)."""
import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs


def bits(v):
    return inputs.f32_to_bf16_bits(np.asarray(v, dtype=np.float32))


def f64(b):
    return inputs.bf16_bits_to_f32(b).astype(np.float64)


def keep_of(x, n, m):
    words = oracle.prune(x, n, m, oracle.MAGNITUDE, want=("mask",))["mask"]
    K = x.shape[1]
    out = np.zeros(x.shape, bool)
    for k in range(K):
        out[:, k] = (words[:, k // 32] >> np.uint32(k % 32)) & np.uint32(1)
    return out


def test_worked_by_hand():
    # two rows, one 2:4 group each (the paper's [1, 7, -3, 2] and a row with ties):
    # kept {7, -3} and {4, first 1}; column sums |x| = [5, 8, 4, 3], kept = [4, 8, 3, 0]
    x = np.zeros((2, 32), np.uint16)
    x[0, :4] = bits([1, 7, -3, 2])
    x[1, :4] = bits([4, 1, 1, 1])
    s = oracle.channel_scales(x, 2, 4)
    assert s[:4].tolist() == [1.25, 1.0, 4.0 / 3.0, 1.0]     # nothing kept in column 3: scale 1
    assert np.all(s[4:] == 1.0)                                # all-zero columns


@pytest.mark.parametrize("n,m", [(2, 4), (1, 4), (2, 8), (2, 16), (4, 8)])
def test_every_channel_keeps_its_l1_norm(n, m):
    x = inputs.relu_masked_laplace_bf16((300, 64), seed=m + n)
    s = oracle.channel_scales(x, n, m)
    keep = keep_of(x, n, m)
    a = np.abs(f64(x))
    total, kept = a.sum(0), (a * keep).sum(0)
    assert np.all(s >= 1.0)
    nz = kept > 0
    np.testing.assert_allclose((a * keep * s).sum(0)[nz], total[nz], rtol=1e-12)   # the defining property
    assert np.all(s[~nz] == 1.0)
    # and not the per-group scales: the channel reading gives ONE factor per column
    np.testing.assert_allclose(s[nz], total[nz] / kept[nz], rtol=1e-12)


def test_nothing_pruned_means_scale_one():
    x = inputs.normal_bf16((50, 64), 1.0, seed=3)
    assert np.all(oracle.channel_scales(x, 4, 4) == 1.0)


def test_single_row_reduces_to_plain_magnitude_pruning():
    # with one row a kept element is its column's whole norm: every scale is 1
    x = inputs.normal_bf16((1, 64), 1.0, seed=4)
    assert np.all(oracle.channel_scales(x, 2, 4) == 1.0)


def test_scaled_contraction_equals_library_matmul_and_weight_folding():
    rng = np.random.default_rng(7)
    x = inputs.relu_masked_laplace_bf16((40, 64), seed=9)
    w = bits(rng.standard_normal((64, 24)) / 8)
    s = oracle.channel_scales(x, 2, 4)
    pruned = oracle.prune(x, 2, 4, oracle.MAGNITUDE, want=("dense",))["dense"]
    got = oracle.dgrad_linear(pruned, w, k_scale=s)
    np.testing.assert_allclose(got, (f64(pruned) * s) @ f64(w), rtol=1e-12, atol=1e-12)
    # the scale may equally be folded into the rows of W: (A diag(s)) W = A (diag(s) W)
    np.testing.assert_allclose(got, f64(pruned) @ (s[:, None] * f64(w)), rtol=1e-12, atol=1e-12)
    assert not np.allclose(got, oracle.dgrad_linear(pruned, w))    # the scales are really applied


def test_scaled_conv_equals_library_transposed_convolution():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(8)
    B, H, Wd, Cin, Cout, R, S, stride, pad = 2, 8, 6, 5, 16, 3, 3, 1, 1
    g = inputs.relu_masked_laplace_bf16((B, H, Wd, Cout), seed=2)
    w = bits(rng.standard_normal((Cout, R, S, Cin)) / 4)
    s = oracle.channel_scales(g.reshape(-1, Cout), 2, 4)
    pruned = oracle.prune(np.pad(g.reshape(-1, Cout), ((0, 0), (0, 16))), 2, 4, oracle.MAGNITUDE, want=("dense",))["dense"][:, :Cout]
    pruned = np.ascontiguousarray(pruned).reshape(g.shape)
    got = oracle.dgrad_conv2d(pruned, w, H, Wd, stride, pad, k_scale=s)
    gt = torch.from_numpy(f64(pruned) * s).permute(0, 3, 1, 2)
    wt = torch.from_numpy(f64(w)).permute(0, 3, 1, 2)
    ref = torch.nn.grad.conv2d_input((B, Cin, H, Wd), wt, gt, stride=stride, padding=pad).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


def test_fp16_element_type():
    x = inputs.bf16_bits_as_f16_bits(inputs.relu_masked_laplace_bf16((64, 32), seed=5))
    s = oracle.channel_scales(x, 2, 4, dtype=oracle.FP16)
    a = np.abs(inputs.f16_bits_to_f32(x).astype(np.float64))
    words = oracle.prune(x, 2, 4, oracle.MAGNITUDE, want=("mask",), dtype=oracle.FP16)["mask"]
    keep = np.array([[(words[r, 0] >> np.uint32(k)) & 1 for k in range(32)] for r in range(64)], bool)
    kept = (a * keep).sum(0)
    np.testing.assert_allclose(s[kept > 0], a.sum(0)[kept > 0] / kept[kept > 0], rtol=1e-12)
