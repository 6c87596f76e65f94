"""Per-channel reading of the L1 rescale on the GPU (SDGP_FLAG_CHANNEL, sdgp_channel_scales) against the
oracle. The factors are fp32 sums combined in no fixed order: compared to 1e-5 relative; dL/dD to the usual
5e-3 relative Frobenius error (the scaled copy of W adds one 16-bit rounding per weight)."""
import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 5e-3


def dev16(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()


def rel_fro(got, ref):
    return np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)


@pytest.mark.parametrize("n,m", [(2, 4), (1, 4), (2, 8), (2, 16), (2, 32), (3, 4), (4, 8), (8, 8)])
@pytest.mark.parametrize("rows,K", [(1000, 128), (37, 64), (3000, 4096), (513, 192)])
def test_channel_scales(rows, K, n, m):
    import paper_2202_00774_b200 as sdgp
    if K % m:
        pytest.skip("K not a multiple of m")
    x = inputs.relu_masked_laplace_bf16((rows, K), seed=K + n + m)
    out = torch.full((3 * K,), -1.0, dtype=torch.float32, device="cuda")
    sdgp.sdgp_channel_scales(dev16(x), n, m, sdgp.BF16, out)
    got = out.cpu().numpy().astype(np.float64)
    want = oracle.channel_scales(x, n, m)
    np.testing.assert_allclose(got[:K], want, rtol=1e-5)
    a = np.abs(inputs.bf16_bits_to_f32(x).astype(np.float64))
    np.testing.assert_allclose(got[K:2 * K], a.sum(0), rtol=1e-5)


def test_channel_scales_fp16_and_empty_columns():
    import paper_2202_00774_b200 as sdgp
    x = inputs.bf16_bits_as_f16_bits(inputs.relu_masked_laplace_bf16((400, 128), seed=3))
    x[:, 5] = 0          # a column of zeros: nothing kept, factor 1
    x[:, 64:68] = inputs.f32_to_f16_bits(np.array([[1.0, 2.0, 3.0, 0.5]], np.float32))   # column 67 never survives 2:4
    out = torch.empty((3 * 128,), dtype=torch.float32, device="cuda")
    sdgp.sdgp_channel_scales(dev16(x), 2, 4, sdgp.FP16, out)
    got = out.cpu().numpy().astype(np.float64)
    want = oracle.channel_scales(x, 2, 4, dtype=oracle.FP16)
    np.testing.assert_allclose(got[:128], want, rtol=1e-5)
    assert got[5] == 1.0 and got[67] == 1.0 and want[67] == 1.0


@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("rows,K,N,n,m", [(333, 512, 128, 2, 4), (1000, 256, 256, 1, 4), (200, 128, 64, 2, 8)])
def test_linear_channel_mode(rows, K, N, n, m, dtype):
    import paper_2202_00774_b200 as sdgp
    dO, W = inputs.fc_tensors(rows, K, N, seed=rows + K)
    # give the channels different magnitudes so the factors differ visibly from column to column
    dO = inputs.f32_to_bf16_bits(inputs.bf16_bits_to_f32(dO) * (1.0 + (np.arange(K) % 7)).astype(np.float32))
    odt, gdt, to_f = oracle.BF16, sdgp.BF16, inputs.bf16_bits_to_f32
    if dtype == "fp16":
        dO, W = inputs.bf16_bits_as_f16_bits(dO), inputs.bf16_bits_as_f16_bits(W)
        odt, gdt, to_f = oracle.FP16, sdgp.FP16, inputs.f16_bits_to_f32
    ws = torch.empty(sdgp.sdgp_workspace_size_linear(rows, K, N, sdgp.FLAG_CHANNEL), dtype=torch.uint8, device="cuda")
    dD = torch.full((rows, N), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_linear_typed(dev16(dO), dev16(W), dD, n, m, sdgp.RESCALED_MAGNITUDE, 0, gdt, workspace=ws,
                                 flags=sdgp.FLAG_CHANNEL)
    assert sdgp.sdgp_last_device_error() == 0
    scales = oracle.channel_scales(dO, n, m, dtype=odt)
    pruned = oracle.prune(dO, n, m, oracle.MAGNITUDE, want=("dense",), dtype=odt)["dense"]
    want = oracle.dgrad_linear(pruned, W, dtype=odt, k_scale=scales)
    got = to_f(dD.cpu().numpy().view(np.uint16)).astype(np.float64)
    assert rel_fro(got, want) <= TOL
    # the per-group scheme and plain magnitude pruning give clearly different results: the mode is really the channel one
    plain = oracle.dgrad_linear(pruned, W, dtype=odt)
    assert rel_fro(plain, want) > 5 * TOL


@pytest.mark.parametrize("case", [(6, 16, 16, 64, 128, 3, 3, 1, 1), (4, 8, 8, 128, 256, 3, 3, 1, 1),
                                  (3, 14, 14, 256, 64, 1, 1, 1, 0), (3, 16, 16, 64, 128, 3, 3, 2, 1)])
def test_conv_channel_mode(case):
    import paper_2202_00774_b200 as sdgp
    B, H, Wd, Cin, Cout, R, S, stride, pad = case
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, stride, pad)
    dO, W = inputs.conv_layer_tensors(layer, seed=Cout + H)
    ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, stride, pad, sdgp.FLAG_CHANNEL),
                     dtype=torch.uint8, device="cuda")
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, stride, pad, 2, 4, sdgp.RESCALED_MAGNITUDE, workspace=ws,
                           flags=sdgp.FLAG_CHANNEL)
    assert sdgp.sdgp_last_device_error() == 0
    flat = dO.reshape(-1, Cout)
    scales = oracle.channel_scales(flat, 2, 4)
    pruned = oracle.prune(flat, 2, 4, oracle.MAGNITUDE, want=("dense",))["dense"].reshape(dO.shape)
    want = oracle.dgrad_conv2d(pruned, W, H, Wd, stride, pad, k_scale=scales)
    got = inputs.bf16_bits_to_f32(dD.cpu().numpy().view(np.uint16)).astype(np.float64)
    assert not np.isnan(got).any()
    assert rel_fro(got, want) <= TOL


def test_channel_mode_wants_the_rescaled_scheme():
    import paper_2202_00774_b200 as sdgp
    dO = torch.zeros((64, 128), dtype=torch.int16, device="cuda")
    W = torch.zeros((128, 64), dtype=torch.int16, device="cuda")
    dD = torch.zeros((64, 64), dtype=torch.int16, device="cuda")
    ws = torch.empty(1 << 18, dtype=torch.uint8, device="cuda")
    with pytest.raises(sdgp.SdgpError) as e:
        sdgp.sdgp_dgrad_linear(dO, W, dD, 2, 4, sdgp.MAGNITUDE, workspace=ws, flags=sdgp.FLAG_CHANNEL)
    assert e.value.status == 1
