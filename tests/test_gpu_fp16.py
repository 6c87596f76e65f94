"""IEEE binary16 tensors through the *_typed entry points, against the oracle's binary16 element type.

Prune outputs are compared bit for bit (ranking reads bit patterns; the rescale's roundings are
fixed); dL/dD within the same relative Frobenius bound as bf16 (binary16 rounds dD more finely)."""
import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 5e-3


def dev16(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()


def host16(t):
    return t.cpu().numpy().view(np.uint16)


def f16_f64(bits):
    return inputs.f16_bits_to_f32(bits).astype(np.float64)


def rel_fro(got, ref):
    return np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)


def fp16_rows(rows, K, seed, adversarial=False):
    if adversarial:
        # binary16 edge patterns: signed zeros, subnormals, largest finite, infinities, NaNs, ties
        g = np.random.Generator(np.random.PCG64([seed, 98]))
        pool = np.array([0x0000, 0x8000, 0x0001, 0x8001, 0x03FF, 0x0400, 0x3C00, 0xBC00, 0x3C00, 0x4000, 0xC000,
                         0x7BFF, 0xFBFF, 0x7C00, 0xFC00, 0x7E00, 0xFE01, 0x3C01, 0xBC01, 0x7800, 0x7A00], dtype=np.uint16)
        return pool[g.integers(0, pool.size, size=(rows, K))]
    return inputs.bf16_bits_as_f16_bits(inputs.relu_masked_laplace_bf16((rows, K), seed))


@pytest.mark.parametrize("adversarial", [False, True])
@pytest.mark.parametrize("scheme", [oracle.RANDOM, oracle.MAGNITUDE, oracle.RESCALED])
@pytest.mark.parametrize("n,m", [(2, 4), (1, 4), (3, 4), (2, 8), (1, 16), (2, 32), (5, 8), (4, 4)])
def test_prune_fp16_bit_exact(n, m, scheme, adversarial):
    import paper_2202_00774_b200 as sdgp
    rows, K = 203, 256   # several blocks and a ragged tail of vectors
    x = fp16_rows(rows, K, seed=n * 7 + m, adversarial=adversarial)
    comp = oracle.compressible(n, m)
    dense = torch.full((rows, K), -1, dtype=torch.int16, device="cuda")
    mask = torch.full((rows, K // 32), -1, dtype=torch.int32, device="cuda")
    values = torch.full((rows, K // 2), -1, dtype=torch.int16, device="cuda") if comp else None
    meta = torch.full((rows, K // 16), -1, dtype=torch.int16, device="cuda") if comp else None
    sdgp.sdgp_prune_typed(dev16(x), n, m, scheme, 77, sdgp.FP16, dense=dense, values=values, meta=meta, mask=mask)
    ref = oracle.prune(x, n, m, scheme, 77, want=("dense", "mask") + (("values", "meta") if comp else ()),
                       dtype=oracle.FP16)
    assert np.array_equal(host16(dense), ref["dense"])
    assert np.array_equal(mask.cpu().numpy().view(np.uint32), ref["mask"])
    if comp:
        assert np.array_equal(host16(values), ref["values"])
        assert np.array_equal(host16(meta), ref["meta"])


@pytest.mark.parametrize("adversarial", [False, True])
@pytest.mark.parametrize("scheme", [oracle.RANDOM, oracle.MAGNITUDE, oracle.RESCALED])
@pytest.mark.parametrize("n,m", [(2, 4), (1, 4), (2, 8), (2, 16)])
def test_prune_fp16_compressed_outputs_alone(n, m, scheme, adversarial):
    """What the two-pass path asks for: values, metadata and mask, no dense copy."""
    import paper_2202_00774_b200 as sdgp
    rows, K = 203, 256
    x = fp16_rows(rows, K, seed=n * 5 + m, adversarial=adversarial)
    mask = torch.full((rows, K // 32), -1, dtype=torch.int32, device="cuda")
    values = torch.full((rows, K // 2), -1, dtype=torch.int16, device="cuda")
    meta = torch.full((rows, K // 16), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_prune_typed(dev16(x), n, m, scheme, 78, sdgp.FP16, values=values, meta=meta, mask=mask)
    ref = oracle.prune(x, n, m, scheme, 78, want=("mask", "values", "meta"), dtype=oracle.FP16)
    assert np.array_equal(host16(values), ref["values"])
    assert np.array_equal(host16(meta), ref["meta"])
    assert np.array_equal(mask.cpu().numpy().view(np.uint32), ref["mask"])


def test_fp16_rescale_differs_from_bf16_rescale_on_the_same_bits():
    # guards against the typed entry point silently running the bf16 arithmetic
    import paper_2202_00774_b200 as sdgp
    x = fp16_rows(64, 128, seed=1)
    a = torch.empty((64, 128), dtype=torch.int16, device="cuda")
    b = torch.empty((64, 128), dtype=torch.int16, device="cuda")
    sdgp.sdgp_prune_typed(dev16(x), 2, 4, sdgp.RESCALED_MAGNITUDE, 0, sdgp.FP16, dense=a)
    sdgp.sdgp_prune_typed(dev16(x), 2, 4, sdgp.RESCALED_MAGNITUDE, 0, sdgp.BF16, dense=b)
    assert not np.array_equal(host16(a), host16(b))


@pytest.mark.parametrize("flags", ["dense", "two_pass", "fused", "masked"])
@pytest.mark.parametrize("rows,K,N", [(333, 512, 128), (130, 256, 256), (77, 128, 64)])
def test_linear_fp16(rows, K, N, flags):
    import paper_2202_00774_b200 as sdgp
    dO_b, W_b = inputs.fc_tensors(rows, K, N, seed=rows)
    dO, W = inputs.bf16_bits_as_f16_bits(dO_b), inputs.bf16_bits_as_f16_bits(W_b)
    dD = torch.full((rows, N), -1, dtype=torch.int16, device="cuda")
    n, m, scheme = (3, 4, oracle.RESCALED) if flags == "masked" else (2, 4, oracle.RESCALED if flags == "two_pass" else oracle.MAGNITUDE)
    flag = {"dense": sdgp.FLAG_DENSE, "two_pass": sdgp.FLAG_TWO_PASS, "fused": sdgp.FLAG_FUSED, "masked": sdgp.FLAG_MASKED}[flags]
    ws = torch.empty(max(16, sdgp.sdgp_workspace_size_linear(rows, K, N, flag)), dtype=torch.uint8, device="cuda")
    sdgp.sdgp_dgrad_linear_typed(dev16(dO), dev16(W), dD, n, m, scheme, 5, sdgp.FP16, workspace=ws, flags=flag)
    assert sdgp.sdgp_last_device_error() == 0
    src = dO if flags == "dense" else oracle.prune(dO, n, m, scheme, 5, want=("dense",), dtype=oracle.FP16)["dense"]
    want = oracle.dgrad_linear(src, W, dtype=oracle.FP16)
    got = f16_f64(host16(dD))
    assert not np.isnan(got).any()
    assert rel_fro(got, want) <= TOL
    # binary16 carries three more fraction bits than bf16: the rounding of dD is well below the bf16 level
    assert rel_fro(got, want) <= 6e-4


@pytest.mark.parametrize("mode", ["dense", "two_pass", "fused_random"])
@pytest.mark.parametrize("case", [(3, 16, 16, 64, 128, 3, 3, 1, 1), (2, 8, 8, 128, 256, 3, 3, 1, 1),
                                  (2, 14, 14, 256, 128, 1, 1, 1, 0), (2, 16, 16, 64, 128, 3, 3, 2, 1),
                                  (5, 32, 32, 64, 128, 3, 3, 1, 1)])
def test_conv_fp16(case, mode):
    import paper_2202_00774_b200 as sdgp
    B, H, Wd, Cin, Cout, R, S, stride, pad = case
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, stride, pad)
    dO_b, W_b = inputs.conv_layer_tensors(layer, seed=H + Cout)
    dO, W = inputs.bf16_bits_as_f16_bits(dO_b), inputs.bf16_bits_as_f16_bits(W_b)
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    if mode == "dense":
        sdgp.sdgp_dgrad_conv2d_typed(dev16(dO), dev16(W), dD, stride, pad, 2, 4, sdgp.MAGNITUDE, 0, sdgp.FP16, flags=sdgp.FLAG_DENSE)
        src = dO
    elif mode == "two_pass":
        ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, stride, pad), dtype=torch.uint8, device="cuda")
        sdgp.sdgp_dgrad_conv2d_typed(dev16(dO), dev16(W), dD, stride, pad, 2, 4, sdgp.RESCALED_MAGNITUDE, 3, sdgp.FP16, workspace=ws)
        src = oracle.prune(dO.reshape(-1, Cout), 2, 4, oracle.RESCALED, 3, want=("dense",), dtype=oracle.FP16)["dense"].reshape(dO.shape)
    else:
        sdgp.sdgp_dgrad_conv2d_typed(dev16(dO), dev16(W), dD, stride, pad, 2, 4, sdgp.RANDOM, 3, sdgp.FP16, flags=sdgp.FLAG_FUSED)
        src = oracle.prune(dO.reshape(-1, Cout), 2, 4, oracle.RANDOM, 3, want=("dense",), dtype=oracle.FP16)["dense"].reshape(dO.shape)
    assert sdgp.sdgp_last_device_error() == 0
    got = f16_f64(host16(dD))
    assert not np.isnan(got).any()
    assert rel_fro(got, oracle.dgrad_conv2d(src, W, H, Wd, stride, pad, dtype=oracle.FP16)) <= 6e-4


def test_spmm_fp16_from_oracle_compressed():
    import paper_2202_00774_b200 as sdgp
    rows, K, N = 300, 256, 128
    dO_b, W_b = inputs.fc_tensors(rows, K, N, seed=8)
    dO, W = inputs.bf16_bits_as_f16_bits(dO_b), inputs.bf16_bits_as_f16_bits(W_b)
    ref = oracle.prune(dO, 2, 8, oracle.MAGNITUDE, want=("dense", "values", "meta"), dtype=oracle.FP16)
    dD = torch.full((rows, N), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_spmm_linear_typed(dev16(ref["values"]), dev16(ref["meta"]), dev16(W), dD, sdgp.FP16)
    assert sdgp.sdgp_last_device_error() == 0
    assert rel_fro(f16_f64(host16(dD)), oracle.dgrad_linear(ref["dense"], W, dtype=oracle.FP16)) <= 6e-4


def test_fp16_requests_without_a_kernel_are_refused():
    import paper_2202_00774_b200 as sdgp
    dO = torch.zeros((64, 128), dtype=torch.int16, device="cuda")
    W = torch.zeros((128, 64), dtype=torch.int16, device="cuda")
    dD = torch.zeros((64, 64), dtype=torch.int16, device="cuda")
    with pytest.raises(sdgp.SdgpError) as e:   # in-kernel prune of the rescaled scheme: bf16 only
        sdgp.sdgp_dgrad_linear_typed(dO, W, dD, 2, 4, sdgp.RESCALED_MAGNITUDE, 0, sdgp.FP16, flags=sdgp.FLAG_FUSED)
    assert e.value.status == 2
    with pytest.raises(sdgp.SdgpError) as e:   # unknown element type
        sdgp.sdgp_dgrad_linear_typed(dO, W, dD, 2, 4, sdgp.MAGNITUDE, 0, 5, flags=sdgp.FLAG_DENSE)
    assert e.value.status == 1
