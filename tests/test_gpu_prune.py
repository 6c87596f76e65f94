"""GPU prune kernel vs the CPU oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a.view(np.int32)).cuda()


def run_gpu(x, n, m, scheme, seed, want_compressed, want_mask=True):
    import paper_2202_00774_b200 as sdgp
    rows, K = x.shape
    d = dev(x)
    dense = torch.full((rows, K), -1, dtype=torch.int16, device="cuda")
    values = torch.full((rows, K // 2), -1, dtype=torch.int16, device="cuda") if want_compressed else None
    meta = torch.full((rows, K // 16), -1, dtype=torch.int16, device="cuda") if want_compressed else None
    mask = torch.full((rows, K // 32), -1, dtype=torch.int32, device="cuda") if want_mask else None
    sdgp.sdgp_prune(d, n, m, scheme, seed, dense=dense, values=values, meta=meta, mask=mask)
    torch.cuda.synchronize()
    out = {"dense": dense.cpu().numpy().view(np.uint16)}
    if want_compressed:
        out["values"] = values.cpu().numpy().view(np.uint16)
        out["meta"] = meta.cpu().numpy().view(np.uint16)
    if want_mask:
        out["mask"] = mask.cpu().numpy().view(np.uint32)
    return out


def compare(x, n, m, scheme, seed=0):
    comp = oracle.compressible(n, m)
    want_mask = x.shape[1] % 32 == 0
    want = ("dense",) + (("values", "meta") if comp else ()) + (("mask",) if want_mask else ())
    ref = oracle.prune(x, n, m, scheme, seed, want=want)
    got = run_gpu(x, n, m, scheme, seed, comp, want_mask)
    for key in want:
        assert np.array_equal(got[key], ref[key]), "%s differs for %d:%d scheme %d" % (key, n, m, scheme)


def compare_compressed_only(x, n, m, scheme, seed=0):
    """The call the two-pass path makes: values and metadata, no dense copy (the rescaled scheme then scales the
    gathered survivors instead of every lane)."""
    import paper_2202_00774_b200 as sdgp
    rows, K = x.shape
    ref = oracle.prune(x, n, m, scheme, seed, want=("values", "meta"))
    values = torch.full((rows, K // 2), -1, dtype=torch.int16, device="cuda")
    meta = torch.full((rows, K // 16), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_prune(dev(x), n, m, scheme, seed, values=values, meta=meta)
    assert np.array_equal(values.cpu().numpy().view(np.uint16), ref["values"]), "values differ for %d:%d scheme %d" % (n, m, scheme)
    assert np.array_equal(meta.cpu().numpy().view(np.uint16), ref["meta"]), "meta differs for %d:%d scheme %d" % (n, m, scheme)


SCHEMES = [oracle.RANDOM, oracle.MAGNITUDE, oracle.RESCALED]
NM = [(1, 4), (2, 4), (3, 4), (4, 4), (1, 8), (2, 8), (4, 8), (2, 16), (5, 16), (2, 32), (4, 32), (16, 32)]


@pytest.mark.parametrize("scheme", SCHEMES)
@pytest.mark.parametrize("n,m", NM)
def test_prune_matches_oracle_ragged(n, m, scheme):
    # 1237 rows x 160: several blocks of 1024 vectors plus a ragged tail
    x = inputs.relu_masked_laplace_bf16((1237, 160), seed=n * 100 + m)
    compare(x, n, m, scheme, seed=0xABCDEF0123 + m)


@pytest.mark.parametrize("scheme", SCHEMES)
@pytest.mark.parametrize("n,m", [(2, 4), (1, 4), (2, 8), (2, 16), (2, 32), (6, 8)])
def test_prune_edge_values(n, m, scheme):
    x = inputs.adversarial_groups_bf16(513, 96, seed=m)  # ties, +-0, Inf, NaN, denormals; K % 32 != 0
    compare(x, n, m, scheme, seed=5)


@pytest.mark.parametrize("rows,K", [(1, 32), (1, 16), (3, 48), (256, 512)])
def test_prune_small_shapes(rows, K):
    x = inputs.normal_bf16((rows, K), 1.0, seed=rows)
    for scheme in SCHEMES:
        compare(x, 2, 4, scheme, seed=1)


def test_prune_empty_is_a_noop():
    import paper_2202_00774_b200 as sdgp
    d = torch.empty((0, 64), dtype=torch.int16, device="cuda")
    sdgp.sdgp_prune(d, 2, 4, sdgp.MAGNITUDE)


def test_prune_does_not_touch_input_or_neighbours():
    import paper_2202_00774_b200 as sdgp
    rows, K = 100, 64
    x = inputs.normal_bf16((rows, K), 1.0, seed=3)
    d = dev(x)
    buf = torch.full((rows * K // 2 + 64,), 0x5A5A, dtype=torch.int16, device="cuda")
    values = buf[32:32 + rows * K // 2].view(rows, K // 2)
    sdgp.sdgp_prune(d, 2, 4, sdgp.MAGNITUDE, values=values, meta=torch.empty((rows, K // 16), dtype=torch.int16, device="cuda"))
    torch.cuda.synchronize()
    assert np.array_equal(d.cpu().numpy().view(np.uint16), x)
    b = buf.cpu().numpy()
    assert np.all(b[:32] == 0x5A5A) and np.all(b[-32:] == 0x5A5A)


def test_prune_full_size_fc_and_sampled_large():
    # the small FC workload in full, and sampled rows of a tensor larger than L2
    x, _ = inputs.fc_tensors(256, 512, 256, seed=0)
    compare(x, 2, 4, oracle.MAGNITUDE)
    big = inputs.relu_masked_laplace_bf16((65536, 1024), seed=9)   # 128 MiB
    for scheme in SCHEMES:
        got = run_gpu(big, 2, 4, scheme, 77, True)
        ref = oracle.prune(big, 2, 4, scheme, 77)
        for key in ("dense", "values", "meta", "mask"):
            assert np.array_equal(got[key], ref[key]), key


@pytest.mark.parametrize("scheme", SCHEMES)
@pytest.mark.parametrize("n,m", [(1, 4), (2, 4), (1, 8), (2, 8), (2, 16), (2, 32)])
def test_prune_compressed_outputs_alone(n, m, scheme):
    compare_compressed_only(inputs.relu_masked_laplace_bf16((1237, 160), seed=n * 10 + m), n, m, scheme, seed=3)
    compare_compressed_only(inputs.adversarial_groups_bf16(513, 96, seed=m + 1), n, m, scheme, seed=4)
