"""Pins for the oracle's random pruning function and its Philox4x32-10 generator."""
import itertools
import os
import subprocess
import sys
import tempfile

import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs
from test_oracle_prune import mask_bits

ENGINE_PROBE = r"""
// Prints 4 raw outputs of an independent open-source Philox4x32-10 engine for each
// "seed subsequence offset" triple on the command line.
#include <ATen/core/PhiloxRNGEngine.h>
#include <cstdio>
#include <cstdlib>
int main(int argc, char** argv) {
  for (int i = 1; i + 2 < argc; i += 3) {
    at::philox_engine e(strtoull(argv[i], 0, 0), strtoull(argv[i + 1], 0, 0), strtoull(argv[i + 2], 0, 0));
    unsigned a = e(), b = e(), c = e(), d = e();
    printf("%u %u %u %u\n", a, b, c, d);
  }
  return 0;
}
"""


def test_philox_matches_independent_engine():
    """The engine header shipped with the installed torch is a separate implementation of the
    same published generator: its counter is (offset_lo, offset_hi, subsequence_lo,
    subsequence_hi) and its key is the seed. The oracle's round function must agree word for word."""
    torch = pytest.importorskip("torch")
    inc = os.path.join(os.path.dirname(torch.__file__), "include")
    if not os.path.exists(os.path.join(inc, "ATen", "core", "PhiloxRNGEngine.h")):
        pytest.skip("engine header not shipped")
    cases = [(0, 0, 0), (1, 0, 0), (0, 1, 0), (0, 0, 1), (5, 7, 9), (0xFFFFFFFFFFFFFFFF, 0, 0xFFFFFFFF),
             (0x0123456789ABCDEF, 0xFEDCBA9876543210, 0x1_0000_0001), (42, 0, 2 ** 40 + 3)]
    with tempfile.TemporaryDirectory() as d:
        src, exe = os.path.join(d, "probe.cpp"), os.path.join(d, "probe")
        with open(src, "w") as f:
            f.write(ENGINE_PROBE)
        subprocess.check_call(["g++", "-std=c++17", "-O1", "-I", inc, src, "-o", exe])
        args = [str(v) for c in cases for v in c]
        lines = subprocess.check_output([exe] + args, text=True).strip().splitlines()
    assert len(lines) == len(cases)
    for (seed, subseq, offset), line in zip(cases, lines):
        want = [int(t) for t in line.split()]
        ctr = [offset & 0xFFFFFFFF, offset >> 32, subseq & 0xFFFFFFFF, subseq >> 32]
        key = [seed & 0xFFFFFFFF, seed >> 32]
        assert oracle.philox4x32_10(ctr, key).tolist() == want


def test_philox_is_a_bijection_on_a_small_slice():
    # distinct counters give distinct outputs (the round function is a permutation of the counter)
    seen = {tuple(oracle.philox4x32_10([c, 0, 0, 0], [3, 4]).tolist()) for c in range(2000)}
    assert len(seen) == 2000


def test_random_key_indexing():
    # element e uses half-word (e & 7) of block e >> 3, counter = block number, key = seed
    seed = 0x1234_5678_9ABC_DEF0
    for e in [0, 1, 7, 8, 9, 1000003, 2 ** 35 + 5]:
        q = e >> 3
        o = oracle.philox4x32_10([q & 0xFFFFFFFF, q >> 32, 0, 0], [seed & 0xFFFFFFFF, seed >> 32])
        half = o.view(np.uint16)  # little-endian half-words
        assert oracle.random_key16(seed, e) == int(half[e & 7])


@pytest.mark.parametrize("n,m", [(2, 4), (1, 4), (2, 8), (4, 16)])
def test_random_mask_is_the_n_smallest_keys(n, m):
    rows, K = 6, 64
    x = inputs.normal_bf16((rows, K), 1.0, seed=1)
    out = oracle.prune(x, n, m, oracle.RANDOM, seed=77, want=("mask",))
    keep = mask_bits(out["mask"], K)
    for r in range(rows):
        for g in range(K // m):
            keys = [(oracle.random_key16(77, r * K + g * m + j), j) for j in range(m)]
            chosen = sorted(j for _, j in sorted(keys)[:n])
            assert np.flatnonzero(keep[r, g * m:(g + 1) * m]).tolist() == chosen


def test_random_mask_depends_on_linear_index_only():
    x = inputs.normal_bf16((8, 256), 1.0, seed=1)
    a = oracle.prune(x, 2, 4, oracle.RANDOM, seed=9, want=("mask",))["mask"]
    b = oracle.prune(x.reshape(16, 128), 2, 4, oracle.RANDOM, seed=9, want=("mask",))["mask"]
    assert np.array_equal(a.reshape(-1), b.reshape(-1))
    # and not on the values
    c = oracle.prune(np.zeros_like(x), 2, 4, oracle.RANDOM, seed=9, want=("mask",))["mask"]
    assert np.array_equal(a, c)
    d = oracle.prune(x, 2, 4, oracle.RANDOM, seed=10, want=("mask",))["mask"]
    assert not np.array_equal(a, d)


@pytest.mark.parametrize("n,m", [(2, 4), (1, 4), (2, 8)])
def test_random_subsets_are_uniform(n, m):
    rows, K = 2048, 512
    x = np.zeros((rows, K), np.uint16)
    keep = mask_bits(oracle.prune(x, n, m, oracle.RANDOM, seed=5, want=("mask",))["mask"], K)
    codes = (keep.reshape(-1, m) * (1 << np.arange(m))).sum(-1)
    subsets = [sum(1 << j for j in s) for s in itertools.combinations(range(m), n)]
    counts = np.array([(codes == s).sum() for s in subsets], dtype=np.float64)
    assert counts.sum() == codes.size  # every group picked a valid n-subset
    expected = codes.size / len(subsets)
    chi2 = ((counts - expected) ** 2 / expected).sum()
    dof = len(subsets) - 1
    assert chi2 < dof + 6 * np.sqrt(2 * dof) + 10


def test_different_seeds_decorrelate():
    x = np.zeros((512, 512), np.uint16)
    a = mask_bits(oracle.prune(x, 2, 4, oracle.RANDOM, seed=1, want=("mask",))["mask"], 512)
    b = mask_bits(oracle.prune(x, 2, 4, oracle.RANDOM, seed=2, want=("mask",))["mask"], 512)
    agree = (a == b).mean()
    assert abs(agree - 0.5) < 0.01


def test_runtime_reduction_closed_form():
    """Section 4.3 numbers, read from the fixture."""
    path = os.path.join(os.path.dirname(__file__), "golden", "runtime_reduction.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        kind, share, n, m, printed = line.split()
        share, n, m, printed = float(share), int(n), int(m), float(printed)
        red = oracle.runtime_reduction(share, n, m)
        got = 100 * red if kind == "reduction" else 100 * (share - red)
        assert abs(got - printed) <= 0.051
