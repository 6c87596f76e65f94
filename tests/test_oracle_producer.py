"""Pins of the oracle's producer of dL/dO (ReLU backward, then Algorithm 1): Section 2.1 / Fig. 2 (dL/dO is what the
layer above hands down), Section 3.1 (the unpruned tensor is kept), Section 3.3 (ReLU zeros)."""
import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs


def bits(values):
    return inputs.f32_to_bf16_bits(np.asarray(values, np.float32))


def test_hand_example():
    # gradient above the ReLU, and the ReLU's activation: positive, zero, negative, negative zero, tiny, NaN, Inf, -Inf
    dY = bits([1.5, -2.0, 3.0, 4.0, -5.0, 6.0, 7.0, -8.0])
    act = np.array([0x3F80, 0x0000, 0xBF80, 0x8000, 0x0001, 0x7FC0, 0x7F80, 0xFF80], np.uint16)
    got = oracle.relu_backward(dY, act)
    want = bits([1.5, 0.0, 0.0, 0.0, -5.0, 0.0, 7.0, 0.0])
    assert np.array_equal(got, want)
    assert got[1] == 0 and got[3] == 0          # blocked positions hold +0.0, not -0.0


def test_equals_the_textbook_derivative_on_random_tensors():
    rng = np.random.default_rng(5)
    for dtype, to_f32 in ((oracle.BF16, inputs.bf16_bits_to_f32),):
        dY = bits(rng.standard_normal((64, 96)))
        act = bits(np.maximum(rng.standard_normal((64, 96)), 0.0))      # a ReLU's output: half exact zeros
        got = oracle.relu_backward(dY, act, dtype)
        want = np.where(to_f32(act) > 0, dY, np.uint16(0))
        assert np.array_equal(got, want)
        # passing the ReLU's INPUT instead of its output selects the same positions
        pre = bits(rng.standard_normal((64, 96)))
        assert np.array_equal(oracle.relu_backward(dY, pre, dtype),
                              oracle.relu_backward(dY, bits(np.maximum(to_f32(pre), 0.0)), dtype))


def test_survivors_keep_their_bits_and_signs():
    dY = np.arange(0, 65536, 7, dtype=np.uint16)[:4096].reshape(64, 64)     # every kind of pattern, NaNs included
    act = np.full(dY.shape, 0x3F80, np.uint16)
    assert np.array_equal(oracle.relu_backward(dY, act), dY)
    assert not oracle.relu_backward(dY, np.zeros_like(dY)).any()


def test_producer_is_relu_backward_followed_by_algorithm_1():
    rng = np.random.default_rng(9)
    dY = bits(rng.laplace(size=(40, 128)))
    act = bits(np.maximum(rng.standard_normal((40, 128)), 0.0))
    for n, m, scheme in ((2, 4, oracle.MAGNITUDE), (1, 4, oracle.RESCALED), (2, 8, oracle.RANDOM), (2, 16, oracle.MAGNITUDE)):
        out = oracle.relu_backward_prune(dY, act, n, m, scheme, seed=3)
        assert np.array_equal(out["grad"], np.where(inputs.bf16_bits_to_f32(act) > 0, dY, np.uint16(0)))
        ref = oracle.prune(out["grad"], n, m, scheme, 3)
        for key in ("dense", "values", "meta", "mask"):
            assert np.array_equal(out[key], ref[key]), key
        # where the ReLU blocks a whole group nothing survives; the pruned copy never holds what the ReLU blocked
        blocked = inputs.bf16_bits_to_f32(act) <= 0
        assert not out["dense"][blocked].any()


def test_worked_example_passes_through_an_open_relu():
    # Section 3.2's example [1, 7, -3, 2] -> [0, 7, -3, 0] with every activation positive
    dY = bits([[1.0, 7.0, -3.0, 2.0] * 4])
    act = bits(np.ones((1, 16)))
    out = oracle.relu_backward_prune(dY, act, 2, 4, oracle.MAGNITUDE, want=("dense",))
    assert np.array_equal(out["dense"], bits([[0.0, 7.0, -3.0, 0.0] * 4]))
    # ... and with the activation of the 7 at zero the 2 takes its place
    act[0, 1] = 0
    out = oracle.relu_backward_prune(dY, act, 2, 4, oracle.MAGNITUDE, want=("dense",))
    assert np.array_equal(out["dense"][0, :4], bits([0.0, 0.0, -3.0, 2.0]))


# ---- the producer below the ReLU that follows a residual addition (the two gradients are added first) ----


def test_residual_sum_hand_examples_of_rounding():
    # bf16 keeps 8 significant bits: 1 + 2^-8 lies exactly between 1 and 1 + 2^-7 and goes to the even one (1);
    # (1 + 2^-7) + 2^-8 lies between 1 + 2^-7 (odd) and 1 + 2^-6 (even) and goes up; 1 + 3 * 2^-9 is above the midpoint
    one, ulp, half_ulp = 0x3F80, 0x3C00, 0x3B80          # 1.0, 2^-7, 2^-8
    act = np.full(8, 0x3F80, np.uint16)
    dY = np.array([one, one + 1, one, 0x4049, 0xC049, 0x7F80, 0x7F80, 0x0000], np.uint16)
    dSkip = np.array([half_ulp, half_ulp, 0x3BC0, 0xC049, 0x4049, 0xFF80, 0x3F80, 0x8000], np.uint16)
    got = oracle.residual_relu_backward(dY, dSkip, act)
    #            tie->even  tie->even(up)  above the tie   x + (-x)  (-x) + x   inf - inf   inf + 1   +0 + -0
    want = np.array([one,    one + 2,       one + 1,        0x0000,   0x0000,    0x7FC0,     0x7F80,   0x0000], np.uint16)
    assert np.array_equal(got, want)
    assert ulp == 0x3C00 and inputs.bf16_bits_to_f32(np.array([one + 1], np.uint16))[0] == 1.0078125


def test_residual_sum_equals_the_libraries_16_bit_addition():
    # torch adds bfloat16 tensors, numpy adds float16 arrays: both libraries round the sum of the two numbers to the
    # 16-bit type, which is what the gradient accumulation of a framework does at a residual connection
    import torch
    rng = np.random.default_rng(11)
    shape = (96, 128)
    act = np.full(shape, 0x3F80, np.uint16)
    for scale in (1.0, 1e-3, 300.0):
        a = bits(rng.standard_normal(shape) * scale)
        b = bits(rng.laplace(size=shape))
        want = (torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) + torch.from_numpy(b.view(np.int16)).view(torch.bfloat16))
        assert np.array_equal(oracle.residual_relu_backward(a, b, act), want.view(torch.int16).numpy().view(np.uint16))
    # every pair of exponents, so that one operand vanishes, half-vanishes or cancels against the other
    a = np.repeat(np.arange(0x0080, 0x7F80, 0x0155, dtype=np.uint16), 64)
    b = np.tile(np.arange(0x8080, 0xFF80, 0x0200, dtype=np.uint16), a.size // 64 + 1)[:a.size]
    want = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) + torch.from_numpy(b.view(np.int16)).view(torch.bfloat16)
    assert np.array_equal(oracle.residual_relu_backward(a, b, np.full(a.shape, 0x3F80, np.uint16)),
                          want.view(torch.int16).numpy().view(np.uint16))
    # binary16
    h = rng.standard_normal(shape).astype(np.float16)
    k = (rng.standard_normal(shape) * 0.01).astype(np.float16)
    got = oracle.residual_relu_backward(h.view(np.uint16), k.view(np.uint16), np.full(shape, 0x3C00, np.uint16), oracle.FP16)
    assert np.array_equal(got, (h + k).view(np.uint16))
    big = np.array([65504.0, 65504.0, -65504.0, 6.1e-5, 5.96e-8], np.float16)        # overflow to infinity, subnormal sums
    small = np.array([32.0, 8.0, -32.0, -6.0e-5, 5.96e-8], np.float16)
    got = oracle.residual_relu_backward(big.view(np.uint16), small.view(np.uint16), np.full(5, 0x3C00, np.uint16), oracle.FP16)
    with np.errstate(over="ignore"):
        assert np.array_equal(got, (big + small).view(np.uint16))


def test_residual_sum_symmetry_gate_and_reduction_to_the_plain_producer():
    rng = np.random.default_rng(12)
    shape = (64, 96)
    dY, dSkip = bits(rng.laplace(size=shape)), bits(rng.laplace(size=shape) * 0.25)
    act = bits(np.maximum(rng.standard_normal(shape), 0.0))
    got = oracle.residual_relu_backward(dY, dSkip, act)
    assert np.array_equal(got, oracle.residual_relu_backward(dSkip, dY, act))           # addition commutes, bit for bit
    blocked = inputs.bf16_bits_to_f32(act) <= 0
    assert blocked.any() and np.all(got[blocked] == 0)
    # the gate is the plain producer's: the sum, formed everywhere, then passed through relu_backward
    everywhere = oracle.residual_relu_backward(dY, dSkip, np.full(shape, 0x3F80, np.uint16))
    assert np.array_equal(got, oracle.relu_backward(everywhere, act))
    # with nothing on the skip path the sum is dY itself (its zeros are +0.0 here)
    assert np.array_equal(oracle.residual_relu_backward(dY, np.zeros(shape, np.uint16), act), oracle.relu_backward(dY, act))
    # an activation that is not a number, negative zero or negative passes nothing
    odd = np.array([0x7FC0, 0x8000, 0xBF80, 0xFF80], np.uint16)
    assert not oracle.residual_relu_backward(dY.ravel()[:4], dSkip.ravel()[:4], odd).any()


def test_residual_producer_is_the_sum_followed_by_algorithm_1():
    rng = np.random.default_rng(13)
    dY, dSkip = bits(rng.laplace(size=(48, 64))), bits(rng.laplace(size=(48, 64)))
    act = bits(np.maximum(rng.standard_normal((48, 64)), 0.0))
    out = oracle.residual_relu_backward_prune(dY, dSkip, act, 2, 4, oracle.MAGNITUDE)
    ref = oracle.prune(out["grad"], 2, 4, oracle.MAGNITUDE)
    for key in ("dense", "values", "meta", "mask"):
        assert np.array_equal(out[key], ref[key])
    f = inputs.bf16_bits_to_f32
    kept = f(out["dense"]) != 0
    assert np.all(f(out["dense"])[kept] == f(out["grad"])[kept]) and kept.reshape(48, 16, 4).sum(-1).max() <= 2


# ---- the producer below a ReLU that is followed by 2 x 2 max pooling (the pooled gradient goes to the window's maximum) ----


def test_maxpool_hand_example():
    # one image of 2 x 4 pixels (two windows), one channel per column of the tables below, K = 4
    f = lambda rows: bits(np.array(rows, np.float32))
    #                 channel: 0 (plain max)  1 (tie: first wins)  2 (nothing positive)  3 (max at the last position)
    act = np.stack([f([[1.0, 2.0, -1.0, 0.5], [3.0, 2.0, 0.0, 0.25]]),        # pixel row 0: window 0 = columns 0, 1
                    f([[2.0, 1.0, -2.0, 0.5], [0.5, 2.0, -0.0, 4.0]])])       # pixel row 1
    act = np.concatenate([act, act[:, ::-1]], axis=1)[None]                   # second window: the first one mirrored left-right
    g = bits(np.array([[[[10.0, 20.0, 30.0, 40.0], [50.0, 60.0, 70.0, 80.0]]]], np.float32))
    got = inputs.bf16_bits_to_f32(oracle.maxpool_relu_backward(g, act))
    want = np.zeros((1, 2, 4, 4), np.float32)
    want[0, 0, 1, 0] = 10.0      # 3.0 at (0, 1)
    want[0, 0, 0, 1] = 20.0      # 2.0 three times: (0, 0) comes first
    want[0, 1, 1, 3] = 40.0      # 4.0 at (1, 1)
    want[0, 0, 2, 0] = 50.0      # mirrored window: 3.0 now at (0, 0) -> pixel column 2
    want[0, 0, 2, 1] = 60.0      # mirrored tie: the first of the three 2.0 is at (0, 0) again
    want[0, 1, 2, 3] = 80.0      # 4.0 now at (1, 0)
    assert np.array_equal(got, want)


def test_maxpool_equals_the_librarys_pooling_and_relu_backward():
    import torch
    rng = np.random.default_rng(21)
    B, H, W, K = 3, 8, 12, 16
    # coarse values, so that equal activations inside a window are common
    pre = bits(np.round(rng.standard_normal((B, H, W, K)) * 2.0) / 2.0)
    g = bits(rng.laplace(size=(B, H // 2, W // 2, K)))
    x = torch.from_numpy(inputs.bf16_bits_to_f32(pre)).double().permute(0, 3, 1, 2).contiguous().requires_grad_(True)
    y = torch.nn.functional.max_pool2d(torch.relu(x), 2)
    y.backward(torch.from_numpy(inputs.bf16_bits_to_f32(g)).double().permute(0, 3, 1, 2).contiguous())
    want = x.grad.permute(0, 2, 3, 1).numpy()
    for act in (pre, bits(np.maximum(inputs.bf16_bits_to_f32(pre), 0.0))):       # the ReLU's input, or its output
        got = oracle.maxpool_relu_backward(g, act)
        assert np.array_equal(inputs.bf16_bits_to_f32(got).astype(np.float64), want)
    ties = (inputs.bf16_bits_to_f32(pre).reshape(B, H // 2, 2, W // 2, 2, K).transpose(0, 1, 3, 5, 2, 4).reshape(-1, 4))
    assert np.any((ties == ties.max(1, keepdims=True)).sum(1) > 1)              # the draw does hold ties


def test_maxpool_invariants_bits_and_special_activations():
    rng = np.random.default_rng(22)
    B, H, W, K = 2, 6, 4, 32
    act = bits(rng.standard_normal((B, H, W, K)))
    flat = act.reshape(-1)
    flat[rng.integers(0, flat.size, 300)] = np.resize(np.array([0x7FC0, 0x7F80, 0x8000, 0x0001, 0xFF80], np.uint16), 300)
    g = np.arange(1, 1 + B * (H // 2) * (W // 2) * K, dtype=np.uint16).reshape(B, H // 2, W // 2, K) * 37     # every kind of pattern
    got = oracle.maxpool_relu_backward(g, act)
    win = got.reshape(B, H // 2, 2, W // 2, 2, K).transpose(0, 1, 3, 5, 2, 4).reshape(B, H // 2, W // 2, K, 4)
    awin = inputs.bf16_bits_to_f32(act).reshape(B, H // 2, 2, W // 2, 2, K).transpose(0, 1, 3, 5, 2, 4).reshape(B, H // 2, W // 2, K, 4)
    with np.errstate(invalid="ignore"):
        positive = awin > 0                                                     # NaN: False
    assert np.all((win != 0).sum(-1) <= 1)
    has = positive.any(-1)
    assert np.array_equal(win.sum(-1, dtype=np.uint32)[has], g[has].astype(np.uint32))     # the survivor is g, bit for bit
    assert not win[~has].any()
    # the survivor sits on a positive activation that no other positive activation of the window exceeds
    sel = win != 0
    cand = np.where(positive, awin, -np.inf)
    assert np.all(cand[sel] == cand.max(-1)[sel.any(-1)])
    # an infinite activation wins its window; a NaN never does
    a = np.full((1, 2, 2, 8), 0x3F80, np.uint16)
    a[0, 1, 0, :] = 0x7F80
    a[0, 0, 0, :] = 0x7FC0
    out = oracle.maxpool_relu_backward(np.full((1, 1, 1, 8), 0x4000, np.uint16), a)
    assert np.all(out[0, 1, 0] == 0x4000) and not out[0, 0].any() and not out[0, 1, 1].any()


def test_maxpool_producer_is_the_scatter_followed_by_algorithm_1():
    rng = np.random.default_rng(23)
    act = bits(rng.standard_normal((2, 4, 4, 64)))
    g = bits(rng.laplace(size=(2, 2, 2, 64)))
    out = oracle.maxpool_relu_backward_prune(g, act, 2, 8, oracle.MAGNITUDE)
    ref = oracle.prune(out["grad"].reshape(-1, 64), 2, 8, oracle.MAGNITUDE)
    for key in ("dense", "values", "meta", "mask"):
        assert np.array_equal(out[key], ref[key])
    with pytest.raises(ValueError):
        oracle.maxpool_relu_backward(g, act[:, :3])                              # odd height


def test_maxpool_producer_with_a_second_gradient_adds_before_it_scatters():
    rng = np.random.default_rng(24)
    act = bits(rng.standard_normal((2, 4, 4, 32)))
    g, k = bits(rng.laplace(size=(2, 2, 2, 32))), bits(rng.laplace(size=(2, 2, 2, 32)) * 0.125)
    out = oracle.maxpool_relu_backward_prune(g, act, 2, 4, oracle.MAGNITUDE, skip=k)
    import torch
    total = (torch.from_numpy(g.view(np.int16)).view(torch.bfloat16) + torch.from_numpy(k.view(np.int16)).view(torch.bfloat16))
    total = total.view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(out["grad"], oracle.maxpool_relu_backward(total, act))
    assert np.array_equal(oracle.maxpool_relu_backward_prune(g, act, 2, 4, oracle.MAGNITUDE, skip=np.zeros_like(g))["grad"],
                          oracle.maxpool_relu_backward(g, act))
