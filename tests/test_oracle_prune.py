"""Pins for the oracle's pruning step (Algorithm 1, Section 3.2).

None of these compare the oracle with itself: they use the example the paper
prints, brute-force enumeration of every kept subset, exact rational
arithmetic, and structural invariants.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(vals):
    return inputs.f32_to_bf16_bits(np.asarray(vals, dtype=np.float32))


def as_f64(b):
    return inputs.bf16_bits_to_f32(b).astype(np.float64)


def mask_bits(mask_words, K):
    """[rows, K/32] u32 -> [rows, K] bool."""
    rows = mask_words.shape[0]
    out = np.zeros((rows, K), bool)
    for k in range(K):
        out[:, k] = (mask_words[:, k // 32] >> np.uint32(k % 32)) & np.uint32(1)
    return out


def prune_small(x_bits, n, m, scheme, seed=0):
    """Oracle on one [rows, K] array whose K may be < 32: pad K up to a multiple of 32
    with whole extra groups, then cut the padding off again."""
    x_bits = np.atleast_2d(x_bits)
    rows, K = x_bits.shape
    Kp = ((K + 31) // 32) * 32
    while Kp % m:
        Kp += 32
    xp = np.zeros((rows, Kp), np.uint16)
    xp[:, :K] = x_bits
    want = ("dense", "mask") + (("values", "meta") if oracle.compressible(n, m) else ())
    out = oracle.prune(xp, n, m, scheme, seed, want=want)
    return out["dense"][:, :K], mask_bits(out["mask"], Kp)[:, :K], out


# ------------------------------------------------------------- paper example


def read_worked_example():
    rows = {}
    with open(os.path.join(GOLDEN, "worked_example_magnitude.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            rows[key] = [float(v) for v in vals]
    return rows


def test_paper_worked_example_magnitude():
    ex = read_worked_example()
    dense, keep, _ = prune_small(bits(ex["input"]), 2, 4, oracle.MAGNITUDE)
    assert as_f64(dense[0]).tolist() == ex["result"]
    # the kept values are the first n of the paper's ranking
    assert sorted(as_f64(dense[0])[keep[0]].tolist()) == sorted(ex["ranked"][:2])


def test_paper_worked_example_rescaled():
    # Same group under the L1-preserving rescale: |1|+|7|+|-3|+|2| = 13, kept 7+3 = 10,
    # so survivors are multiplied by 13/10 and rounded to bf16 (spacing 1/16 near 9, 1/64 near 3.9).
    ex = read_worked_example()
    dense, _, _ = prune_small(bits(ex["input"]), 2, 4, oracle.RESCALED)
    assert as_f64(dense[0]).tolist() == [0.0, 9.125, -3.90625, 0.0]


# --------------------------------------------------------------- brute force


def brute_force_keep(x, n):
    """Among all n-subsets: largest magnitudes first (compare the descending-sorted
    magnitude vectors lexicographically); equal vectors -> the smallest index tuple."""
    m = len(x)
    best = None
    for sub in itertools.combinations(range(m), n):
        score = tuple(sorted((abs(x[j]) for j in sub), reverse=True))
        cand = (score, tuple(-j for j in sub))
        if best is None or cand > best[0]:
            best = (cand, sub)
    keep = np.zeros(m, bool)
    keep[list(best[1])] = True
    return keep


@pytest.mark.parametrize("n", [1, 2, 3, 4])
def test_magnitude_brute_force_exhaustive_m4(n):
    vals = [-2.0, -1.0, 0.0, 1.0, 2.0]
    groups = np.array(list(itertools.product(vals, repeat=4)), dtype=np.float32)  # 625 groups, many ties
    x = bits(groups)
    _, keep, _ = prune_small(x.reshape(1, -1), n, 4, oracle.MAGNITUDE)
    keep = keep.reshape(-1, 4)
    for g in range(groups.shape[0]):
        assert np.array_equal(keep[g], brute_force_keep(groups[g].tolist(), n)), (groups[g], n)


@pytest.mark.parametrize("m,n", [(8, 1), (8, 2), (8, 3), (8, 5), (8, 8), (4, 2), (16, 2)])
def test_magnitude_brute_force_random(m, n):
    rng = np.random.default_rng(m * 100 + n)
    # few distinct magnitudes -> frequent ties; includes exact zeros and both signs
    groups = rng.integers(-3, 4, size=(300 if m < 16 else 60, m)).astype(np.float32) * 0.5
    x = bits(groups)
    _, keep, _ = prune_small(x.reshape(1, -1), n, m, oracle.MAGNITUDE)
    keep = keep.reshape(-1, m)
    for g in range(groups.shape[0]):
        assert np.array_equal(keep[g], brute_force_keep(groups[g].tolist(), n))


# ---------------------------------------------------------------- invariants


@pytest.mark.parametrize("scheme", [oracle.RANDOM, oracle.MAGNITUDE, oracle.RESCALED])
@pytest.mark.parametrize("n,m", [(1, 4), (2, 4), (2, 8), (2, 16), (4, 8), (4, 32), (16, 32), (3, 4), (4, 4)])
def test_structure_exactly_n_kept_per_group(scheme, n, m):
    x = inputs.relu_masked_laplace_bf16((64, 128), seed=3)
    out = oracle.prune(x, n, m, scheme, seed=11, want=("dense", "mask"))
    keep = mask_bits(out["mask"], 128)
    assert np.all(keep.reshape(64, 128 // m, m).sum(-1) == n)
    # pruned slots are +0.0 (bit pattern 0), never -0.0
    assert np.all(out["dense"][~keep] == 0)
    if scheme != oracle.RESCALED:
        assert np.array_equal(out["dense"][keep], x[keep])  # survivors keep their exact bits


@pytest.mark.parametrize("n,m", [(2, 4), (2, 8), (1, 4), (4, 16), (8, 32)])
def test_magnitude_survivors_dominate_pruned(n, m):
    x = inputs.adversarial_groups_bf16(50, 128, seed=5)  # NaN, Inf, -0.0, denormals, ties
    out = oracle.prune(x, n, m, oracle.MAGNITUDE, want=("mask",))
    keep = mask_bits(out["mask"], 128).reshape(50, -1, m)
    key = (x & 0x7FFF).astype(np.int64).reshape(50, -1, m)
    kept_min = np.where(keep, key, 1 << 20).min(-1)
    pruned_max = np.where(~keep, key, -1).max(-1)
    assert np.all(kept_min >= pruned_max)
    # ties go to the lower index: a pruned element equal to the smallest kept key
    # must sit after every kept element with that key
    idx = np.arange(m)
    for r in range(50):
        for g in range(keep.shape[1]):
            k, kp = key[r, g], keep[r, g]
            t = kept_min[r, g]
            tied_pruned = idx[(~kp) & (k == t)]
            tied_kept = idx[kp & (k == t)]
            if tied_pruned.size and tied_kept.size:
                assert tied_kept.max() < tied_pruned.min()


def test_half_zero_groups_keep_zero_elements():
    # With many exact zeros a kept element may itself be zero: n kept, at most n nonzero.
    x = bits([[0, 0, 0, 5, 0, 0, 0, 0] * 4])
    dense, keep, _ = prune_small(x, 2, 4, oracle.MAGNITUDE)
    assert keep[0, :8].tolist() == [True, False, False, True, True, True, False, False]
    assert np.count_nonzero(dense[0, :4]) == 1


# ------------------------------------------------------------------ rescale


@pytest.mark.parametrize("n,m", [(1, 4), (2, 4), (2, 8), (2, 16), (4, 32), (3, 8)])
def test_rescale_same_mask_and_l1_preserved(n, m):
    x = inputs.relu_masked_laplace_bf16((40, 128), seed=8)
    mag = oracle.prune(x, n, m, oracle.MAGNITUDE, want=("dense", "mask"))
    res = oracle.prune(x, n, m, oracle.RESCALED, want=("dense", "mask"))
    assert np.array_equal(mag["mask"], res["mask"])  # Section 3.3: same elements pruned
    xv = as_f64(x).reshape(40, -1, m)
    yv = as_f64(res["dense"]).reshape(40, -1, m)
    mv = as_f64(mag["dense"]).reshape(40, -1, m)
    assert np.all(np.sign(yv) == np.sign(mv))
    l1_in, l1_out, l1_kept = np.abs(xv).sum(-1), np.abs(yv).sum(-1), np.abs(mv).sum(-1)
    nz = l1_kept > 0
    # ||group||_1 is preserved up to one bf16 rounding per survivor
    assert np.all(np.abs(l1_out[nz] - l1_in[nz]) <= 2.0 ** -7 * l1_in[nz])
    scale = l1_out[nz] / l1_kept[nz]
    assert np.all(scale >= 1 - 2.0 ** -7) and np.all(scale <= m / n * (1 + 2.0 ** -7))
    # groups of all zeros stay all zeros
    assert np.all(l1_out[~nz] == 0)


def test_rescale_matches_exact_rational_within_one_rounding():
    """Every survivor equals x * (sum|group| / sum|kept|) computed exactly, up to the fp32
    and bf16 roundings the method allows (2^-8 bf16 half-ulp bound plus fp32 slack)."""
    rng = np.random.default_rng(21)
    x = bits(rng.standard_normal((200, 32)).astype(np.float32))
    for n, m in [(2, 4), (2, 8), (1, 4), (5, 16)]:
        res = oracle.prune(x, n, m, oracle.RESCALED, want=("dense", "mask"))
        keep = mask_bits(res["mask"], 32)
        for r in range(0, 200, 7):
            for g in range(32 // m):
                sl = slice(g * m, (g + 1) * m)
                xs = [Fraction(float(v)) for v in as_f64(x[r, sl])]
                T = sum(abs(v) for v in xs)
                S = sum(abs(v) for v, k in zip(xs, keep[r, sl]) if k)
                for j in range(m):
                    y = Fraction(float(as_f64(res["dense"][r, sl])[j]))
                    if not keep[r, sl][j]:
                        assert y == 0
                    else:
                        exact = xs[j] * T / S
                        assert abs(y - exact) <= abs(exact) * Fraction(1, 256) * Fraction(1001, 1000)


def test_rescale_exact_cases():
    # power-of-two scales are exact in every precision involved
    dense, _, _ = prune_small(bits([[3, 1, 1, 1]]), 1, 4, oracle.RESCALED)
    assert as_f64(dense[0]).tolist() == [6.0, 0, 0, 0]              # 6/3 = 2
    dense, _, _ = prune_small(bits([[-3, 1, 1, 1]]), 2, 4, oracle.RESCALED)
    assert as_f64(dense[0]).tolist() == [-4.5, 1.5, 0, 0]          # 6/4 = 1.5, tie -> index 1
    dense, _, _ = prune_small(bits([[2, -2, 2, -2, 0, 0, 0, 0]]), 2, 8, oracle.RESCALED)
    assert as_f64(dense[0]).tolist() == [4.0, -4.0, 0, 0, 0, 0, 0, 0]  # 8/4 = 2
    dense, _, _ = prune_small(bits([[0, 0, 0, 0]]), 2, 4, oracle.RESCALED)
    assert dense[0].tolist() == [0, 0, 0, 0]                           # zero denominator: scale 1


@pytest.mark.parametrize("m", [4, 8, 16, 32])
def test_rescale_identity_when_nothing_is_pruned(m):
    x = inputs.normal_bf16((16, 64), 1.0, seed=2)
    res = oracle.prune(x, m, m, oracle.RESCALED, want=("dense",))
    assert np.array_equal(res["dense"], x)  # T == S -> scale exactly 1
    # ... also for groups that hold Inf or NaN: with nothing pruned there is nothing to rescale
    # (Section 3.2 rescales "the remaining n elements" of a group that lost m - n), so no Inf/Inf arises
    y = inputs.adversarial_groups_bf16(16, 64, seed=4)
    res = oracle.prune(y, m, m, oracle.RESCALED, want=("dense",))
    assert np.array_equal(res["dense"], y)


# ---------------------------------------------------------- compressed form


VALID_NIBBLES = {p0 | (p1 << 2) for p0 in range(4) for p1 in range(p0 + 1, 4)}


@pytest.mark.parametrize("scheme", [oracle.RANDOM, oracle.MAGNITUDE, oracle.RESCALED])
@pytest.mark.parametrize("n,m", [(1, 4), (2, 4), (2, 8), (2, 16), (1, 8), (2, 32)])
def test_compressed_round_trip(scheme, n, m):
    x = inputs.relu_masked_laplace_bf16((33, 96 if m != 32 else 128), seed=4)
    K = x.shape[1]
    out = oracle.prune(x, n, m, scheme, seed=7, want=("dense", "values", "meta"))
    assert out["values"].shape == (33, K // 2) and out["meta"].shape == (33, K // 16)
    assert np.array_equal(oracle.expand(out["values"], out["meta"]), out["dense"])
    nibs = np.stack([(out["meta"] >> (4 * i)) & 0xF for i in range(4)], -1)
    assert set(np.unique(nibs).tolist()) <= VALID_NIBBLES


def test_compressed_examples_by_hand():
    # survivors {1,2} -> slots (x1, x2), nibble 1 | 2<<2 = 9
    # survivors {3}   -> padded with position 0: slots (0, x3), nibble 0 | 3<<2 = 12
    # survivors {0}   -> padded with position 1: slots (x0, 0), nibble 0 | 1<<2 = 4
    # no nonzero at all under 1:4 keeps position 0 (tie-break) -> nibble 4, both slots zero-valued
    x = bits([[1, 7, -3, 2, 0.5, 0.25, 0.125, 9, 5, 0, 0, 0, 0, 0, 0, 0]])
    o24 = oracle.prune(x, 2, 4, oracle.MAGNITUDE, want=("values", "meta"))
    assert as_f64(o24["values"][0]).tolist() == [7, -3, 0.5, 9, 5, 0, 0, 0]
    assert o24["meta"][0, 0] == (9 | (12 << 4) | (4 << 8) | (4 << 12))
    o14 = oracle.prune(x, 1, 4, oracle.MAGNITUDE, want=("values", "meta"))
    assert as_f64(o14["values"][0]).tolist() == [0, 7, 0, 9, 5, 0, 0, 0]
    assert o14["meta"][0, 0] == ((0 | 1 << 2) | ((0 | 3 << 2) << 4) | (4 << 8) | (4 << 12))


def test_incompressible_patterns_are_rejected():
    x = inputs.normal_bf16((4, 64), 1.0, seed=1)
    with pytest.raises(ValueError):
        oracle.prune(x, 4, 8, oracle.MAGNITUDE, want=("values", "meta"))
    with pytest.raises(ValueError):
        oracle.prune(x, 2, 6, oracle.MAGNITUDE, want=("dense",))  # 64 % 6 != 0
    with pytest.raises(ValueError):
        oracle.prune(x, 5, 4, oracle.MAGNITUDE, want=("dense",))
    with pytest.raises(ValueError):
        oracle.prune(x, 2, 64, oracle.MAGNITUDE, want=("dense",))  # m > 32


# --------------------------------------------------------- planted mistakes


def test_pins_catch_a_wrong_tie_break():
    """A ranking that broke ties toward the higher index would disagree with brute force
    on the groups used above (sanity check that the pins have teeth)."""
    x = [1.0, 1.0, 1.0, 1.0]
    assert brute_force_keep(x, 2).tolist() == [True, True, False, False]
    _, keep, _ = prune_small(bits([x]), 2, 4, oracle.MAGNITUDE)
    assert keep[0].tolist() == [True, True, False, False]
