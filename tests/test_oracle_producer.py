"""Pins of the oracle's producer of dL/dO (ReLU backward, then Algorithm 1): Section 2.1 / Fig. 2 (dL/dO is what the
layer above hands down), Section 3.1 (the unpruned tensor is kept), Section 3.3 (ReLU zeros)."""
import numpy as np

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
