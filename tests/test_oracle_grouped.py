"""Pins for the oracle's data gradient of a grouped convolution (the 3x3 convolutions of RegNetX, Section 4;
the contraction itself is Section 2.1, Fig. 2 and Fig. 3)."""
import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs

torch = pytest.importorskip("torch")


def f64(b):
    return inputs.bf16_bits_to_f32(b).astype(np.float64)


def rel_fro(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def tensors(B, H, Wd, Cin, Cout, R, S, stride, pad, groups, seed):
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, stride, pad, groups)
    return inputs.conv_layer_tensors(layer, seed)


def block_diagonal(W, groups):
    """The same filters as an ordinary convolution's W [Cout,R,S,Cin]: zeros outside each group's own block."""
    Cout, R, S, cin_g = W.shape
    cout_g = Cout // groups
    full = np.zeros((Cout, R, S, cin_g * groups), np.uint16)
    for g in range(groups):
        full[g * cout_g:(g + 1) * cout_g, :, :, g * cin_g:(g + 1) * cin_g] = W[g * cout_g:(g + 1) * cout_g]
    return full


CASES = [
    # B, H, W, Cin, Cout, R, S, stride, pad, groups
    (2, 6, 5, 8, 8, 3, 3, 1, 1, 2),
    (1, 7, 7, 12, 24, 3, 3, 1, 1, 3),      # more output than input channels per group
    (2, 8, 8, 32, 16, 3, 3, 2, 1, 4),      # stride 2, fewer output channels per group
    (1, 9, 6, 20, 20, 3, 3, 2, 1, 10),     # two channels per group, odd height
    (1, 5, 5, 6, 6, 1, 1, 1, 0, 6),        # depthwise 1x1
    (1, 6, 6, 16, 16, 2, 3, 1, 1, 2),      # filter that is not square
]


@pytest.mark.parametrize("B,H,Wd,Cin,Cout,R,S,stride,pad,groups", CASES)
def test_equals_library_transposed_convolution(B, H, Wd, Cin, Cout, R, S, stride, pad, groups):
    dO, W = tensors(B, H, Wd, Cin, Cout, R, S, stride, pad, groups, seed=11)
    got = oracle.dgrad_conv2d_grouped(dO, W, H, Wd, groups, stride, pad)
    g = torch.from_numpy(f64(dO)).permute(0, 3, 1, 2).contiguous()
    w = torch.from_numpy(f64(W)).permute(0, 3, 1, 2).contiguous()                 # [Cout, Cin/groups, R, S]
    want = torch.nn.grad.conv2d_input((B, Cin, H, Wd), w, g, stride=stride, padding=pad, groups=groups)
    assert rel_fro(got, want.permute(0, 2, 3, 1).numpy()) < 1e-14


@pytest.mark.parametrize("B,H,Wd,Cin,Cout,R,S,stride,pad,groups", CASES)
def test_equals_the_ordinary_gradient_with_block_diagonal_filters(B, H, Wd, Cin, Cout, R, S, stride, pad, groups):
    dO, W = tensors(B, H, Wd, Cin, Cout, R, S, stride, pad, groups, seed=12)
    got = oracle.dgrad_conv2d_grouped(dO, W, H, Wd, groups, stride, pad)
    want = oracle.dgrad_conv2d(dO, block_diagonal(W, groups), H, Wd, stride, pad)
    assert np.array_equal(got, want)        # the extra terms are exact zeros


def test_one_group_is_the_ordinary_convolution():
    dO, W = tensors(2, 6, 6, 16, 32, 3, 3, 1, 1, 1, seed=13)
    assert np.array_equal(oracle.dgrad_conv2d_grouped(dO, W, 6, 6, 1, 1, 1), oracle.dgrad_conv2d(dO, W, 6, 6, 1, 1))


def test_each_group_is_a_convolution_of_its_own():
    B, H, Wd, Cin, Cout, groups = 2, 6, 7, 24, 48, 3
    dO, W = tensors(B, H, Wd, Cin, Cout, 3, 3, 1, 1, groups, seed=14)
    got = oracle.dgrad_conv2d_grouped(dO, W, H, Wd, groups, 1, 1)
    ci, co = Cin // groups, Cout // groups
    for g in range(groups):
        part = oracle.dgrad_conv2d(np.ascontiguousarray(dO[..., g * co:(g + 1) * co]), W[g * co:(g + 1) * co], H, Wd, 1, 1)
        assert np.array_equal(got[..., g * ci:(g + 1) * ci], part)


def test_groups_do_not_mix():
    B, H, Wd, Cin, Cout, groups = 1, 5, 5, 16, 16, 4
    dO, W = tensors(B, H, Wd, Cin, Cout, 3, 3, 1, 1, groups, seed=15)
    base = oracle.dgrad_conv2d_grouped(dO, W, H, Wd, groups, 1, 1)
    changed = dO.copy()
    changed[..., 4:8] ^= np.uint16(0x8000)                      # flip the sign of group 1's gradient
    got = oracle.dgrad_conv2d_grouped(changed, W, H, Wd, groups, 1, 1)
    assert np.array_equal(got[..., 4:8], -base[..., 4:8])
    keep = np.r_[0:4, 8:16]
    assert np.array_equal(got[..., keep], base[..., keep])


def test_one_hot_filter_routes_a_channel_within_its_group():
    # W[co, 1, 1, cj] = 1 for one (co, cj): dD channel g*cin_g + cj is dO channel co, everything else is zero
    B, H, Wd, Cin, Cout, groups = 1, 4, 4, 8, 8, 2
    dO, _ = tensors(B, H, Wd, Cin, Cout, 3, 3, 1, 1, groups, seed=16)
    W = np.zeros((Cout, 3, 3, Cin // groups), np.uint16)
    W[6, 1, 1, 3] = 0x3F80                                      # output channel 6 (group 1), its input channel 3 -> dD channel 7
    got = oracle.dgrad_conv2d_grouped(dO, W, H, Wd, groups, 1, 1)
    assert np.array_equal(got[..., 7], f64(dO[..., 6]))
    assert not got[..., :7].any()


def test_pixel_subset_and_pruned_input():
    B, H, Wd, Cin, Cout, groups = 2, 8, 8, 32, 32, 2
    dO, W = tensors(B, H, Wd, Cin, Cout, 3, 3, 2, 1, groups, seed=17)
    pruned = oracle.prune(dO.reshape(-1, Cout), 2, 4, oracle.MAGNITUDE, want=("dense",))["dense"].reshape(dO.shape)
    full = oracle.dgrad_conv2d_grouped(pruned, W, H, Wd, groups, 2, 1)
    idx = np.array([0, 5, 63, 64, 127], np.int64)
    assert np.array_equal(oracle.dgrad_conv2d_grouped(pruned, W, H, Wd, groups, 2, 1, pixel_index=idx),
                          full.reshape(-1, Cin)[idx])


def test_rejects_channel_counts_the_groups_do_not_divide():
    dO = np.zeros((1, 4, 4, 6), np.uint16)
    W = np.zeros((6, 3, 3, 2), np.uint16)
    with pytest.raises(ValueError):
        oracle.dgrad_conv2d_grouped(dO, W, 4, 4, 4, 1, 1)      # 6 output channels, 4 groups


def test_regnetx_shape_set():
    layers = inputs.regnetx_400mf_layers(2)
    grouped = [l for l in layers if l.groups > 1]
    assert sorted({(l.Cin, l.groups) for l in grouped}) == [(32, 2), (64, 4), (160, 10), (384, 24)]
    assert all(l.Cin // l.groups == 16 and l.Cout // l.groups == 16 for l in grouped)
    assert all(l.P * l.stride == l.H for l in layers)
