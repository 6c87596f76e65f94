"""Pins for the oracle's IEEE binary16 element type (the precision the paper trained in, Section 4).

The element type enters the method in two places only: where the rescale of Section 3.2 reads
values as numbers and rounds the survivors, and in the contraction. Pinned here against numpy's
float16 (an independent implementation of the format), exact rational arithmetic, the paper's
worked example and library fp64 routines; ranking is shown to be the same integer order.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs


def f16_bits(vals):
    return np.asarray(vals, dtype=np.float32).astype(np.float16).view(np.uint16)


def f16_f64(b):
    return np.ascontiguousarray(b, dtype=np.uint16).view(np.float16).astype(np.float64)


def mask_bits(mask_words, K):
    rows = mask_words.shape[0]
    out = np.zeros((rows, K), bool)
    for k in range(K):
        out[:, k] = (mask_words[:, k // 32] >> np.uint32(k % 32)) & np.uint32(1)
    return out


# ---------------------------------------------------------------- the format


def test_every_binary16_pattern_widens_exactly():
    allbits = np.arange(65536, dtype=np.uint16)
    want = allbits.view(np.float16).astype(np.float64)
    got = np.array([oracle.f16_to_f64(int(b)) for b in allbits])
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))   # -0.0 keeps its sign


def test_round_to_nearest_even_matches_numpy():
    rng = np.random.default_rng(5)
    # random fp32 bit patterns (all exponents, subnormals of both formats, overflow range)
    u = rng.integers(0, 2 ** 32, size=60000, dtype=np.uint64).astype(np.uint32)
    x = u.view(np.float32)
    # exact halfway cases between neighbouring binary16 values, and their fp32 neighbours
    h = rng.integers(0, 0x7BFF, size=4000).astype(np.uint16)
    lo, hi = h.view(np.float16).astype(np.float32), (h + 1).astype(np.uint16).view(np.float16).astype(np.float32)
    mid = ((lo.astype(np.float64) + hi.astype(np.float64)) / 2).astype(np.float32)   # exact in fp32
    ties = np.concatenate([mid, np.nextafter(mid, np.float32(np.inf)), np.nextafter(mid, np.float32(-np.inf)), -mid])
    edge = np.array([0.0, -0.0, 65504.0, 65519.996, 65520.0, 65536.0, 1e10, -1e10, 2.0 ** -24, 2.0 ** -25,
                     np.nextafter(np.float32(2.0 ** -25), np.float32(1)), 2.0 ** -14, np.inf, -np.inf], dtype=np.float32)
    for arr in (x, ties, edge):
        finite_or_inf = ~np.isnan(arr)
        with np.errstate(over="ignore"):
            want = arr.astype(np.float16).view(np.uint16)
        got = np.array([oracle.f32_to_f16(float(v)) for v in arr], dtype=np.uint16)
        assert np.array_equal(got[finite_or_inf], want[finite_or_inf])
    assert oracle.f32_to_f16(float("nan")) == 0x7E00    # the one canonical quiet NaN


def test_magnitude_rank_is_the_integer_order_of_the_cleared_sign_pattern():
    # for finite binary16 values |a| < |b| <=> (bits_a & 0x7FFF) < (bits_b & 0x7FFF)
    pos = np.arange(0x7C01, dtype=np.uint16)           # +0 ... +inf
    vals = pos.view(np.float16).astype(np.float64)
    assert np.all(np.diff(vals) > 0)


# ------------------------------------------------------------------- pruning


def test_paper_worked_example_in_fp16():
    # Section 3.2: [1, 7, -3, 2] keeps 7 and -3; rescaled by 13/10: 9.1 -> 9.1015625 (spacing 2^-7
    # near 9), -3.9 -> -3.900390625 (spacing 2^-9 near 3.9)
    x = np.zeros((1, 32), np.uint16)
    x[0, :4] = f16_bits([1, 7, -3, 2])
    mag = oracle.prune(x, 2, 4, oracle.MAGNITUDE, want=("dense",), dtype=oracle.FP16)["dense"]
    assert f16_f64(mag[0, :4]).tolist() == [0.0, 7.0, -3.0, 0.0]
    res = oracle.prune(x, 2, 4, oracle.RESCALED, want=("dense",), dtype=oracle.FP16)["dense"]
    assert f16_f64(res[0, :4]).tolist() == [0.0, 9.1015625, -3.900390625, 0.0]


@pytest.mark.parametrize("scheme", [oracle.MAGNITUDE, oracle.RANDOM])
@pytest.mark.parametrize("n,m", [(2, 4), (2, 8), (4, 16)])
def test_selection_does_not_depend_on_the_element_type(n, m, scheme):
    # ranking only reads bit patterns: the same bits give the same mask and the same survivors
    x = np.random.default_rng(m).integers(0, 65536, size=(32, 64), dtype=np.uint64).astype(np.uint16)
    a = oracle.prune(x, n, m, scheme, 9, want=("dense", "mask"), dtype=oracle.BF16)
    b = oracle.prune(x, n, m, scheme, 9, want=("dense", "mask"), dtype=oracle.FP16)
    assert np.array_equal(a["mask"], b["mask"]) and np.array_equal(a["dense"], b["dense"])


def test_rescale_fp16_matches_exact_rational_within_one_rounding():
    rng = np.random.default_rng(33)
    x = f16_bits(rng.standard_normal((120, 32)) * 4)
    for n, m in [(2, 4), (1, 4), (2, 8), (5, 16)]:
        res = oracle.prune(x, n, m, oracle.RESCALED, want=("dense", "mask"), dtype=oracle.FP16)
        mag = oracle.prune(x, n, m, oracle.MAGNITUDE, want=("mask",), dtype=oracle.FP16)
        assert np.array_equal(res["mask"], mag["mask"])
        keep = mask_bits(res["mask"], 32)
        for r in range(0, 120, 5):
            for g in range(32 // m):
                sl = slice(g * m, (g + 1) * m)
                xs = [Fraction(float(v)) for v in f16_f64(x[r, sl])]
                T = sum(abs(v) for v in xs)
                S = sum(abs(v) for v, k in zip(xs, keep[r, sl]) if k)
                for j in range(m):
                    y = Fraction(float(f16_f64(res["dense"][r, sl])[j]))
                    if not keep[r, sl][j]:
                        assert y == 0
                    else:
                        exact = xs[j] * T / S
                        # half an ulp of binary16 (2^-11 relative) plus fp32 slack
                        assert abs(y - exact) <= abs(exact) * Fraction(1, 2048) * Fraction(1001, 1000)


def test_rescale_fp16_exact_and_overflow_cases():
    def run(vals, n, m):
        x = np.zeros((1, 32), np.uint16)
        x[0, :len(vals)] = f16_bits(vals)
        return f16_f64(oracle.prune(x, n, m, oracle.RESCALED, want=("dense",), dtype=oracle.FP16)["dense"][0, :len(vals)]).tolist()
    assert run([3, 1, 1, 1], 1, 4) == [6.0, 0, 0, 0]
    assert run([-3, 1, 1, 1], 2, 4) == [-4.5, 1.5, 0, 0]
    assert run([0, 0, 0, 0], 2, 4) == [0, 0, 0, 0]
    # 60000 * (4 * 60000 / 60000) overflows binary16: IEEE rounding gives infinity
    assert run([60000, 60000, 60000, 60000], 1, 4) == [np.inf, 0, 0, 0]
    # subnormal inputs are ordinary numbers: 4 x 2^-24 kept as one element of 2^-22
    assert run([2.0 ** -24] * 4, 1, 4) == [2.0 ** -22, 0, 0, 0]


# --------------------------------------------------------------- contraction


def test_fp16_linear_equals_library_matmul():
    rng = np.random.default_rng(3)
    a = f16_bits(rng.standard_normal((37, 96)))
    w = f16_bits(rng.standard_normal((96, 24)) / 8)
    got = oracle.dgrad_linear(a, w, dtype=oracle.FP16)
    np.testing.assert_allclose(got, f16_f64(a) @ f16_f64(w), rtol=1e-12, atol=1e-12)
    # the same bits read as bf16 are different numbers: the element type really is used
    assert not np.allclose(got, oracle.dgrad_linear(a, w, dtype=oracle.BF16))


def test_fp16_conv_equals_library_transposed_convolution():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(4)
    B, H, Wd, Cin, Cout, R, S, stride, pad = 2, 9, 7, 5, 8, 3, 3, 2, 1
    P, Q = (H + 2 * pad - R) // stride + 1, (Wd + 2 * pad - S) // stride + 1
    g = f16_bits(rng.standard_normal((B, P, Q, Cout)))
    w = f16_bits(rng.standard_normal((Cout, R, S, Cin)) / 4)
    got = oracle.dgrad_conv2d(g, w, H, Wd, stride, pad, dtype=oracle.FP16)
    gt = torch.from_numpy(f16_f64(g)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(f16_f64(w)).permute(0, 3, 1, 2)
    ref = torch.nn.grad.conv2d_input((B, Cin, H, Wd), wt, gt, stride=stride, padding=pad).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


def test_unknown_element_type_is_rejected():
    x = np.zeros((1, 32), np.uint16)
    with pytest.raises(ValueError):
        oracle.prune(x, 2, 4, oracle.MAGNITUDE, dtype=7)
