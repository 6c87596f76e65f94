"""GPU data-gradient kernels vs the fp64 CPU oracle, through the C ABI.

Tolerance: relative Frobenius error <= 5e-3 against the fp64 result computed from the same
pruned bf16 inputs (fp32 accumulation plus one bf16 rounding per output sits near 2e-3). A norm alone
would let a few wholly wrong rows through, so the full-tensor cases also bound EVERY element:
|got - ref| <= 2^-7 |ref| + 2^-16 sum_k |a_k| |b_k|  (one rounding to bf16, relative 2^-8, with a factor two
to spare; fp32 accumulation of up to a few thousand products, each step off by at most 2^-24 of the
running magnitude, again with room to spare). The second term comes from the oracle run on the operands'
magnitudes."""
import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 5e-3


def dev16(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()


def to_f64(t):
    return inputs.bf16_bits_to_f32(t.cpu().numpy().view(np.uint16)).astype(np.float64)


def rel_fro(got, ref):
    return np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)


def magnitudes(bits):
    """The same 16-bit patterns with the sign cleared."""
    return (np.asarray(bits).view(np.uint16) & np.uint16(0x7FFF)).astype(np.uint16)


def assert_close(got, want, absdot=None, what=""):
    """Norm bound, and - when the oracle's sum of |a||b| per output is given - the bound on every element."""
    assert rel_fro(got, want) <= TOL, what
    if absdot is not None:
        bound = 2.0 ** -7 * np.abs(want) + 2.0 ** -16 * absdot
        bad = np.abs(got - want) > bound
        assert not bad.any(), "%s: %d elements off, first at %s" % (what, int(bad.sum()), np.argwhere(bad)[0])


def linear_ref(src, W):
    return oracle.dgrad_linear(src, W), oracle.dgrad_linear(magnitudes(src), magnitudes(W))


def conv_ref(src, W, H, Wd, stride, pad, **kw):
    return (oracle.dgrad_conv2d(src, W, H, Wd, stride, pad, **kw),
            oracle.dgrad_conv2d(magnitudes(src), magnitudes(W), H, Wd, stride, pad, **kw))


def check_no_device_error():
    import paper_2202_00774_b200 as sdgp
    assert sdgp.sdgp_last_device_error() == 0


# ------------------------------------------------------------------- linear


@pytest.mark.parametrize("rows,K,N", [(256, 512, 256), (300, 256, 128), (77, 128, 64), (1000, 384, 192), (128, 64, 64)])
def test_dense_linear(rows, K, N):
    import paper_2202_00774_b200 as sdgp
    dO, W = inputs.fc_tensors(rows, K, N, seed=rows)
    dD = torch.full((rows, N), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_linear(dev16(dO), dev16(W), dD, 4, 4, sdgp.MAGNITUDE, flags=sdgp.FLAG_DENSE)
    check_no_device_error()
    assert_close(to_f64(dD), *linear_ref(dO, W))


@pytest.mark.parametrize("rows,K,N", [(256, 512, 256), (300, 256, 128), (77, 128, 64), (1000, 384, 192)])
def test_spmm_linear_from_oracle_compressed(rows, K, N):
    """The contraction alone: feed the oracle's compressed tensors to the sparse kernel."""
    import paper_2202_00774_b200 as sdgp
    dO, W = inputs.fc_tensors(rows, K, N, seed=rows + 1)
    ref = oracle.prune(dO, 2, 4, oracle.MAGNITUDE, want=("dense", "values", "meta"))
    dD = torch.full((rows, N), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_spmm_linear(dev16(ref["values"]), dev16(ref["meta"]), dev16(W), dD)
    check_no_device_error()
    assert_close(to_f64(dD), *linear_ref(ref["dense"], W))


@pytest.mark.parametrize("scheme", [oracle.RANDOM, oracle.MAGNITUDE, oracle.RESCALED])
@pytest.mark.parametrize("n,m", [(2, 4), (1, 4), (2, 8), (2, 16), (2, 32), (4, 4)])
def test_pruned_linear_two_pass(n, m, scheme):
    import paper_2202_00774_b200 as sdgp
    rows, K, N = 333, 512, 128
    dO, W = inputs.fc_tensors(rows, K, N, seed=n + m)
    ws = torch.empty(sdgp.sdgp_workspace_size_linear(rows, K, N), dtype=torch.uint8, device="cuda")
    dD = torch.full((rows, N), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_linear(dev16(dO), dev16(W), dD, n, m, scheme, seed=42, workspace=ws)
    check_no_device_error()
    pruned = oracle.prune(dO, n, m, scheme, 42, want=("dense",))["dense"]
    assert_close(to_f64(dD), *linear_ref(pruned, W))


# Patterns with more than two survivors in some aligned 4-chunk have no 2:4 form: the masked mode
# prunes into a dense copy and contracts it on the dense pipe (Algorithm 1 as printed; Section 4.2's
# sparsity sweep 4:8 ... 16:32).
@pytest.mark.parametrize("scheme", [oracle.RANDOM, oracle.MAGNITUDE, oracle.RESCALED])
@pytest.mark.parametrize("n,m", [(3, 4), (4, 8), (4, 16), (8, 16), (4, 32), (16, 32), (2, 4), (8, 8)])
def test_pruned_linear_masked(n, m, scheme):
    import paper_2202_00774_b200 as sdgp
    rows, K, N = 301, 384, 192
    dO, W = inputs.fc_tensors(rows, K, N, seed=3 * n + m)
    ws = torch.empty(sdgp.sdgp_workspace_size_linear(rows, K, N, sdgp.FLAG_MASKED), dtype=torch.uint8, device="cuda")
    dD = torch.full((rows, N), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_linear(dev16(dO), dev16(W), dD, n, m, scheme, seed=17, workspace=ws, flags=sdgp.FLAG_MASKED)
    check_no_device_error()
    pruned = oracle.prune(dO, n, m, scheme, 17, want=("dense",))["dense"]
    # the workspace holds Algorithm 1's return value, bit for bit (n == m prunes nothing: dO is read directly)
    assert n == m or np.array_equal(ws.cpu().numpy()[:rows * K * 2].view(np.uint16).reshape(rows, K), pruned)
    assert_close(to_f64(dD), *linear_ref(pruned, W))


@pytest.mark.parametrize("n,m,scheme", [(4, 8, oracle.MAGNITUDE), (3, 4, oracle.RESCALED), (8, 32, oracle.RANDOM)])
@pytest.mark.parametrize("case", [(3, 16, 16, 64, 128, 3, 3, 1, 1), (2, 14, 14, 128, 64, 1, 1, 1, 0),
                                  (2, 15, 13, 64, 128, 3, 3, 2, 1), (5, 8, 8, 128, 256, 3, 3, 1, 1)])
def test_pruned_conv_masked(case, n, m, scheme):
    import paper_2202_00774_b200 as sdgp
    B, H, Wd, Cin, Cout, R, S, stride, pad = case
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, stride, pad)
    dO, W = inputs.conv_layer_tensors(layer, seed=n + Cout)
    ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, stride, pad, sdgp.FLAG_MASKED),
                     dtype=torch.uint8, device="cuda")
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, stride, pad, n, m, scheme, seed=23, workspace=ws, flags=sdgp.FLAG_MASKED)
    check_no_device_error()
    pruned = oracle.prune(dO.reshape(-1, Cout), n, m, scheme, 23, want=("dense",))["dense"].reshape(dO.shape)
    assert_close(to_f64(dD), *conv_ref(pruned, W, H, Wd, stride, pad))


def test_sparse_modes_refuse_patterns_without_a_2_4_form():
    import paper_2202_00774_b200 as sdgp
    dO = torch.zeros((64, 128), dtype=torch.int16, device="cuda")
    W = torch.zeros((128, 64), dtype=torch.int16, device="cuda")
    dD = torch.zeros((64, 64), dtype=torch.int16, device="cuda")
    ws = torch.empty(1 << 16, dtype=torch.uint8, device="cuda")
    for flags in (sdgp.FLAG_TWO_PASS, sdgp.FLAG_FUSED):
        with pytest.raises(sdgp.SdgpError) as e:
            sdgp.sdgp_dgrad_linear(dO, W, dD, 4, 8, sdgp.MAGNITUDE, workspace=ws, flags=flags)
        assert e.value.status == 2


def test_fc_small_config_full():
    """The single-FC workload: dO [256,512], W [512,256], 2:4 magnitude, seed 0."""
    import paper_2202_00774_b200 as sdgp
    c = inputs.FC_SMALL
    dO, W = inputs.fc_tensors(c["rows"], c["K"], c["N"], c["seed"])
    ws = torch.empty(sdgp.sdgp_workspace_size_linear(c["rows"], c["K"], c["N"]), dtype=torch.uint8, device="cuda")
    dD = torch.empty((c["rows"], c["N"]), dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_linear(dev16(dO), dev16(W), dD, 2, 4, sdgp.MAGNITUDE, workspace=ws)
    check_no_device_error()
    pruned = oracle.prune(dO, 2, 4, oracle.MAGNITUDE, want=("dense",))["dense"]
    assert_close(to_f64(dD), *linear_ref(pruned, W))


# --------------------------------------------------------------------- conv


CONV_CASES = [
    # B, H, W, Cin, Cout, R, S, pad
    (3, 8, 8, 64, 128, 3, 3, 1),
    (2, 16, 16, 128, 128, 3, 3, 1),
    (5, 4, 4, 64, 256, 3, 3, 1),      # several images per tile, ragged batch
    (1, 32, 32, 64, 128, 3, 3, 1),
    (2, 14, 14, 64, 128, 1, 1, 0),    # 1x1, image width not a power of two
    (3, 7, 7, 128, 128, 3, 3, 1),
    (1, 10, 12, 64, 128, 3, 3, 0),    # no padding: output grid smaller than input grid
    (1, 9, 9, 64, 128, 5, 5, 2),
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_dense_conv(case):
    import paper_2202_00774_b200 as sdgp
    B, H, Wd, Cin, Cout, R, S, pad = case
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, 1, pad)
    dO, W = inputs.conv_layer_tensors(layer, seed=H)
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, 1, pad, 4, 4, sdgp.MAGNITUDE, flags=sdgp.FLAG_DENSE)
    check_no_device_error()
    assert_close(to_f64(dD), *conv_ref(dO, W, H, Wd, 1, pad))


@pytest.mark.parametrize("scheme", [oracle.RANDOM, oracle.MAGNITUDE, oracle.RESCALED])
@pytest.mark.parametrize("case", CONV_CASES)
def test_pruned_conv_two_pass(case, scheme):
    import paper_2202_00774_b200 as sdgp
    B, H, Wd, Cin, Cout, R, S, pad = case
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, 1, pad)
    dO, W = inputs.conv_layer_tensors(layer, seed=H + 1)
    ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, 1, pad), dtype=torch.uint8,
                     device="cuda")
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, 1, pad, 2, 4, scheme, seed=7, workspace=ws)
    check_no_device_error()
    pruned = oracle.prune(dO.reshape(-1, Cout), 2, 4, scheme, 7, want=("dense",))["dense"].reshape(dO.shape)
    assert_close(to_f64(dD), *conv_ref(pruned, W, H, Wd, 1, pad))


# Shapes that switch on the kernel's shared-memory reuse modes: enough tiles that every CTA
# pair gets several (resident W), 3x3 filters on 16- and 32-wide images (one A image serves the
# three vertical taps), 64 input channels (32-column W halves), two channel blocks (streamed W).
REUSE_CASES = [
    (40, 16, 16, 128, 128, 3, 3, 1),
    (20, 32, 32, 64, 128, 3, 3, 1),
    (40, 16, 16, 128, 256, 3, 3, 1),
    (3, 32, 32, 192, 128, 3, 3, 1),
    (80, 8, 8, 64, 128, 3, 3, 1),
    (24, 16, 16, 64, 64, 3, 3, 1),
]


@pytest.mark.parametrize("mode", ["dense", "sparse"])
@pytest.mark.parametrize("case", REUSE_CASES)
def test_conv_reuse_modes_sampled(case, mode):
    import paper_2202_00774_b200 as sdgp
    B, H, Wd, Cin, Cout, R, S, pad = case
    if mode == "sparse" and Cout % 128:
        pytest.skip("compressed path needs Cout % 128 == 0")
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, 1, pad)
    dO, W = inputs.conv_layer_tensors(layer, seed=B + Cin)
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    if mode == "dense":
        sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, 1, pad, 4, 4, sdgp.MAGNITUDE, flags=sdgp.FLAG_DENSE)
        src = dO
    else:
        ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, 1, pad), dtype=torch.uint8,
                         device="cuda")
        sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, 1, pad, 2, 4, sdgp.MAGNITUDE, seed=3, workspace=ws)
        src = oracle.prune(dO.reshape(-1, Cout), 2, 4, oracle.MAGNITUDE, 3, want=("dense",))["dense"].reshape(dO.shape)
    check_no_device_error()
    rng = np.random.default_rng(1)
    npix = B * H * Wd
    idx = np.unique(np.concatenate([rng.integers(0, npix, 1500), np.arange(0, 300), np.arange(npix - 300, npix)]))
    got = to_f64(dD).reshape(npix, Cin)[idx]
    assert_close(got, *conv_ref(src, W, H, Wd, 1, pad, pixel_index=idx))
    # nothing outside the sample is left unwritten (the buffer was pre-filled with 0xFFFF = NaN)
    assert not np.isnan(to_f64(dD)).any()


STRIDE2_CASES = [
    # B, H, W, Cin, Cout, R, S, pad      (stride 2)
    (3, 16, 16, 64, 128, 3, 3, 1),
    (2, 28, 28, 128, 128, 3, 3, 1),     # bottleneck 3x3 / 2
    (2, 14, 14, 64, 128, 1, 1, 0),      # 1x1 / 2 projection: three of four output parities are zero
    (2, 15, 13, 64, 128, 3, 3, 1),      # odd sizes: parity classes of different extent
    (1, 12, 12, 64, 128, 5, 5, 2),
]


@pytest.mark.parametrize("mode", ["dense", "sparse"])
@pytest.mark.parametrize("case", STRIDE2_CASES)
def test_conv_stride2(case, mode):
    import paper_2202_00774_b200 as sdgp
    B, H, Wd, Cin, Cout, R, S, pad = case
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, 2, pad)
    dO, W = inputs.conv_layer_tensors(layer, seed=H + Cin)
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    if mode == "dense":
        sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, 2, pad, 4, 4, sdgp.MAGNITUDE, flags=sdgp.FLAG_DENSE)
        src = dO
    else:
        ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, 2, pad), dtype=torch.uint8,
                         device="cuda")
        sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, 2, pad, 2, 4, sdgp.RESCALED_MAGNITUDE, seed=3, workspace=ws)
        src = oracle.prune(dO.reshape(-1, Cout), 2, 4, oracle.RESCALED, 3, want=("dense",))["dense"].reshape(dO.shape)
    check_no_device_error()
    got = to_f64(dD)
    assert not np.isnan(got).any()
    assert_close(got, *conv_ref(src, W, H, Wd, 2, pad))


# Output-channel counts that are not whole 128-channel blocks: the compressed rows are padded.
PADDED_CASES = [
    (2, 14, 14, 64, 64, 3, 3, 1, 1),     # B, H, W, Cin, Cout, R, S, stride, pad
    (2, 14, 14, 256, 64, 1, 1, 1, 0),
    (2, 8, 8, 64, 192, 3, 3, 1, 1),
    (2, 16, 16, 64, 64, 3, 3, 2, 1),
]


@pytest.mark.parametrize("scheme", [oracle.MAGNITUDE, oracle.RANDOM])
@pytest.mark.parametrize("case", PADDED_CASES)
def test_pruned_conv_partial_channel_block(case, scheme):
    import paper_2202_00774_b200 as sdgp
    B, H, Wd, Cin, Cout, R, S, stride, pad = case
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, stride, pad)
    dO, W = inputs.conv_layer_tensors(layer, seed=Cout)
    ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, stride, pad), dtype=torch.uint8,
                     device="cuda")
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, stride, pad, 2, 4, scheme, seed=11, workspace=ws)
    check_no_device_error()
    pruned = oracle.prune(dO.reshape(-1, Cout), 2, 4, scheme, 11, want=("dense",))["dense"].reshape(dO.shape)
    assert_close(to_f64(dD), *conv_ref(pruned, W, H, Wd, stride, pad))


def test_resnet50_bottleneck_shapes_small_batch():
    """Every distinct stride-1 bottleneck convolution of ResNet-50 (batch 2), 2:4 magnitude."""
    import paper_2202_00774_b200 as sdgp
    for layer in inputs.resnet50_stride1_layers(batch=2):
        dO, W = inputs.conv_layer_tensors(layer, seed=layer.Cin + layer.Cout)
        ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(layer.B, layer.H, layer.W, layer.Cin, layer.Cout, layer.R,
                                                         layer.S, 1, layer.pad), dtype=torch.uint8, device="cuda")
        dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
        sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, 1, layer.pad, 2, 4, sdgp.MAGNITUDE, workspace=ws)
        check_no_device_error()
        pruned = oracle.prune(dO.reshape(-1, layer.Cout), 2, 4, oracle.MAGNITUDE, 0, want=("dense",))["dense"]
        rng = np.random.default_rng(layer.Cin)
        idx = np.unique(rng.integers(0, layer.B * layer.H * layer.W, 400))
        want = oracle.dgrad_conv2d(pruned.reshape(dO.shape), W, layer.H, layer.W, 1, layer.pad, pixel_index=idx)
        got = to_f64(dD).reshape(-1, layer.Cin)[idx]
        assert rel_fro(got, want) <= TOL, layer.name


def test_resnet18_shapes_small_batch():
    """Every distinct convolution of the ResNet-18 stages (batch 3; stride-2 3x3 and 1x1 shortcuts included),
    2:4 magnitude two-pass, all outputs against the oracle."""
    import paper_2202_00774_b200 as sdgp
    for layer in inputs.resnet18_layers(batch=3):
        dO, W = inputs.conv_layer_tensors(layer, seed=layer.Cin + layer.H)
        ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(layer.B, layer.H, layer.W, layer.Cin, layer.Cout, layer.R,
                                                         layer.S, layer.stride, layer.pad), dtype=torch.uint8, device="cuda")
        dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
        sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, layer.stride, layer.pad, 2, 4, sdgp.MAGNITUDE, workspace=ws)
        check_no_device_error()
        pruned = oracle.prune(dO.reshape(-1, layer.Cout), 2, 4, oracle.MAGNITUDE, 0, want=("dense",))["dense"]
        rng = np.random.default_rng(layer.Cout)
        idx = np.unique(np.concatenate([rng.integers(0, layer.B * layer.H * layer.W, 500), np.arange(0, 60)]))
        want = oracle.dgrad_conv2d(pruned.reshape(dO.shape), W, layer.H, layer.W, layer.stride, layer.pad, pixel_index=idx)
        got_all = to_f64(dD)
        assert not np.isnan(got_all).any(), layer.name
        assert rel_fro(got_all.reshape(-1, layer.Cin)[idx], want) <= TOL, layer.name


def test_memory_bound_1x1_layer_cold_inputs_repeated():
    """A 1x1 convolution with many short tiles per CTA (ResNet-50 128->512 at 28 x 28, batch 256) launched again and
    again with its inputs flushed from L2 in between: operand boxes then arrive late and out of request order,
    which the stage hand-over between the loader, the metadata warps and the MMA thread must tolerate.
    The tensors are drawn on the device (same law as the other convolution inputs); sampled rows go to the oracle."""
    import paper_2202_00774_b200 as sdgp
    B, HW, Cin, Cout = 256, 28, 128, 512
    rows = B * HW * HW
    g = torch.Generator(device="cuda").manual_seed(5)
    u = torch.rand((rows, Cout), generator=g, device="cuda") - 0.5
    lap = -torch.sign(u) * torch.log1p(-2 * u.abs())                       # Laplace(0, 1)
    lap[torch.rand((rows, Cout), generator=g, device="cuda") < 0.5] = 0.0   # ReLU zeros
    dO = lap.to(torch.bfloat16).view(torch.int16)
    del u, lap
    W = (torch.randn((Cout, Cin), generator=g, device="cuda") * (2.0 / Cin) ** 0.5).to(torch.bfloat16).view(torch.int16)
    vals = torch.empty((rows, Cout // 2), dtype=torch.int16, device="cuda")
    meta = torch.empty((rows, Cout // 16), dtype=torch.int16, device="cuda")
    dD = torch.full((B, HW, HW, Cin), -1, dtype=torch.int16, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    sdgp.sdgp_prune(dO, 2, 4, sdgp.MAGNITUDE, 0, values=vals, meta=meta)
    for _ in range(25):
        flush.zero_()
        sdgp.sdgp_spmm_conv2d(vals.view(B, HW, HW, Cout // 2), meta.view(B, HW, HW, Cout // 16), W.view(Cout, 1, 1, Cin), dD, 1, 0)
        sdgp.sdgp_spmm_conv2d(vals.view(B, HW, HW, Cout // 2), meta.view(B, HW, HW, Cout // 16), W.view(Cout, 1, 1, Cin), dD, 1, 0)
    torch.cuda.synchronize()
    check_no_device_error()
    idx = torch.from_numpy(np.unique(np.concatenate([np.random.default_rng(2).integers(0, rows, 400), [0, rows - 1]]))).cuda()
    sample = dO[idx].cpu().numpy().view(np.uint16)
    pruned = oracle.prune(sample, 2, 4, oracle.MAGNITUDE, want=("dense",))["dense"]
    want = oracle.dgrad_linear(pruned, W.cpu().numpy().view(np.uint16))
    got = to_f64(dD.view(rows, Cin)[idx])
    assert rel_fro(got, want) <= TOL
    assert not np.isnan(to_f64(dD)).any()


# ------------------------------------------------------------------- fused


FUSED_CASES = [
    # B, H, W, Cin, Cout, R, S, stride, pad
    (1, 1, 333, 128, 512, 1, 1, 1, 0),      # fully connected
    (1, 1, 1000, 256, 256, 1, 1, 1, 0),
    (3, 8, 8, 64, 128, 3, 3, 1, 1),
    (40, 16, 16, 128, 128, 3, 3, 1, 1),     # filter-row reuse + resident W
    (6, 32, 32, 64, 128, 3, 3, 1, 1),
    (2, 14, 14, 64, 64, 3, 3, 1, 1),        # half a channel block
    (2, 16, 16, 64, 128, 3, 3, 2, 1),       # stride 2
    (2, 16, 16, 128, 256, 3, 3, 1, 1),      # two channel blocks
]


@pytest.mark.parametrize("scheme,n", [(oracle.MAGNITUDE, 2), (oracle.RESCALED, 2), (oracle.RANDOM, 2), (oracle.MAGNITUDE, 1),
                                      (oracle.RANDOM, 1)])
@pytest.mark.parametrize("case", FUSED_CASES)
def test_fused_prune_and_dgrad(case, scheme, n):
    """SDGP_FLAG_FUSED: no workspace; the kernel prunes dense dL/dO itself (groups of 4)."""
    import paper_2202_00774_b200 as sdgp
    B, H, Wd, Cin, Cout, R, S, stride, pad = case
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, stride, pad)
    dO, W = inputs.conv_layer_tensors(layer, seed=B + Cout)
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, stride, pad, n, 4, scheme, seed=21, flags=sdgp.FLAG_FUSED)
    check_no_device_error()
    pruned = oracle.prune(dO.reshape(-1, Cout), n, 4, scheme, 21, want=("dense",))["dense"].reshape(dO.shape)
    got = to_f64(dD)
    assert not np.isnan(got).any()
    assert_close(got, *conv_ref(pruned, W, H, Wd, stride, pad))


# Shapes for the whole-filter-reuse kernel (more than one tap, images at least one 8 x 16 strip
# large): ragged strips in both directions, one and two strips per tile set, odd strip counts,
# wide filters, non-square filters, missing padding, two channel blocks, a half-empty last channel
# block, 64 / 128 / 256 input channels, stride 2 (parity classes with 1 x 2, 2 x 1 and 2 x 2 taps).
HALO_CASES = [
    # B, H, W, Cin, Cout, R, S, stride, pad
    (3, 20, 24, 64, 128, 3, 3, 1, 1),
    (2, 16, 8, 128, 128, 3, 3, 1, 1),       # a single strip per image
    (5, 12, 40, 64, 64, 3, 3, 1, 1),        # five strips: the last tile set has one
    (2, 17, 17, 128, 256, 3, 3, 1, 1),
    (1, 24, 24, 64, 128, 5, 5, 1, 2),
    (2, 16, 16, 64, 128, 1, 3, 1, 0),       # one filter row, no padding
    (2, 16, 16, 64, 128, 3, 1, 1, 0),       # one filter column, no padding
    (3, 16, 16, 256, 128, 3, 3, 1, 1),      # 256 input channels: one strip per tile set
    (2, 16, 16, 128, 192, 3, 3, 1, 1),      # second channel block half empty
    (2, 32, 32, 64, 128, 3, 3, 2, 1),       # stride 2 on 32 x 32: 16 x 16 parity classes
    (2, 28, 28, 128, 128, 3, 3, 1, 1),
    (9, 16, 16, 128, 128, 3, 3, 1, 1),      # odd number of tile sets: a pair with one phantom set
    (168, 16, 16, 64, 64, 3, 3, 1, 1),      # 84 pair tiles on 74 CTA pairs: the last round is dealt out strip by strip
    (5, 8, 8, 256, 128, 3, 3, 1, 1),        # images 8 pixels tall: a strip is 8 rows of TWO images; odd batch
    (4, 8, 16, 64, 128, 3, 3, 1, 1),        # the same with two strips side by side
    (3, 6, 8, 128, 128, 3, 3, 1, 1),        # 6 pixel rows: two of the strip's eight are padding
    (2, 8, 8, 64, 128, 5, 5, 1, 2),         # 5 x 5 filter on 8 x 8 images
    (6, 8, 8, 128, 256, 3, 3, 1, 1),        # two channel blocks
    (16, 4, 4, 512, 512, 3, 3, 1, 1),       # images 4 pixels wide: two per strip row, a box per filter column
    (8, 4, 4, 64, 128, 3, 3, 1, 1),         # ... two strips (four images) per box row
    (6, 4, 4, 128, 128, 3, 3, 1, 1),        # ... six images: the tile set of eight is partly empty
    (4, 3, 4, 64, 128, 3, 3, 1, 1),         # ... three pixel rows
    (10, 4, 4, 64, 128, 5, 5, 1, 2),        # ... 5 x 5 filter
    (8, 8, 8, 64, 128, 3, 3, 2, 1),         # stride 2 on 8 x 8: 4 x 4 parity classes written through strided views
    (3, 15, 15, 64, 128, 3, 3, 2, 1),       # stride 2 on 15 x 15: a class of 7 rows reads all 8 rows of dL/dO
    (2, 14, 14, 128, 128, 3, 3, 1, 1),      # 14 columns under two strips of 8
    (2, 12, 16, 64, 128, 3, 3, 1, 1),       # 12 rows under a strip of 16
    (3, 16, 16, 64, 128, 3, 3, 1, 0),       # no padding: dL/dO is 14 x 14 and the box starts two pixels inside it
    (3, 7, 8, 64, 128, 3, 3, 1, 1),         # 7 rows of two images
    (5, 16, 16, 64, 128, 3, 3, 1, 2),       # padding 2: dL/dO is 18 x 18, larger than the image
]


@pytest.mark.parametrize("mode", ["dense", "two_pass", "fused", "fused_random", "fused_rescaled_1"])
@pytest.mark.parametrize("case", HALO_CASES)
def test_whole_filter_reuse_kernel(case, mode):
    import paper_2202_00774_b200 as sdgp
    B, H, Wd, Cin, Cout, R, S, stride, pad = case
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, stride, pad)
    dO, W = inputs.conv_layer_tensors(layer, seed=H * 100 + Wd)
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    n, scheme = 2, oracle.MAGNITUDE
    if mode == "dense":
        sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, stride, pad, 4, 4, sdgp.MAGNITUDE, flags=sdgp.FLAG_DENSE)
        src = dO
    else:
        if mode == "fused_random":
            scheme = oracle.RANDOM
        if mode == "fused_rescaled_1":
            n, scheme = 1, oracle.RESCALED
        if mode == "two_pass":
            ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(B, H, Wd, Cin, Cout, R, S, stride, pad), dtype=torch.uint8,
                             device="cuda")
            sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, stride, pad, n, 4, scheme, seed=3, workspace=ws)
        else:
            sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, stride, pad, n, 4, scheme, seed=3, flags=sdgp.FLAG_FUSED)
        src = oracle.prune(dO.reshape(-1, Cout), n, 4, scheme, 3, want=("dense",))["dense"].reshape(dO.shape)
    check_no_device_error()
    got = to_f64(dD)
    assert not np.isnan(got).any()           # every output was written
    assert_close(got, *conv_ref(src, W, H, Wd, stride, pad))


@pytest.mark.parametrize("n,m,scheme", [(2, 8, oracle.MAGNITUDE), (1, 8, oracle.RESCALED), (2, 16, oracle.MAGNITUDE),
                                        (2, 16, oracle.RANDOM), (2, 8, oracle.RANDOM), (1, 16, oracle.RESCALED)])
@pytest.mark.parametrize("case", [(3, 16, 16, 64, 128, 3, 3, 1, 1),      # whole-filter-reuse kernel, two strips
                                  (5, 8, 8, 256, 128, 3, 3, 1, 1),       # ... strips of two images
                                  (2, 16, 16, 128, 256, 3, 3, 1, 1),     # two channel blocks
                                  (5, 4, 4, 64, 256, 3, 3, 1, 1),        # general kernel, several images per tile
                                  (1, 1, 333, 128, 512, 1, 1, 1, 0),     # fully connected
                                  (2, 14, 14, 64, 128, 1, 1, 1, 0)])     # 1 x 1
def test_fused_groups_of_8_and_16(case, n, m, scheme):
    """SDGP_FLAG_FUSED for groups larger than four (n <= 2): the in-kernel prune finds the group's two largest
    keys; a group's vectors sit in one thread or in neighbouring lanes."""
    import paper_2202_00774_b200 as sdgp
    B, H, Wd, Cin, Cout, R, S, stride, pad = case
    layer = inputs.ConvLayer("t", B, H, Wd, Cin, Cout, R, S, stride, pad)
    dO, W = inputs.conv_layer_tensors(layer, seed=B + Cout + m)
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, stride, pad, n, m, scheme, seed=31, flags=sdgp.FLAG_FUSED)
    check_no_device_error()
    pruned = oracle.prune(dO.reshape(-1, Cout), n, m, scheme, 31, want=("dense",))["dense"].reshape(dO.shape)
    got = to_f64(dD)
    assert not np.isnan(got).any()
    assert_close(got, *conv_ref(pruned, W, H, Wd, stride, pad))


def test_fused_groups_of_32():
    """Groups of 32 span four lanes of the whole-filter-reuse kernel's pruning warps; the general kernel (whose
    threads hold 16 channels) refuses them."""
    import paper_2202_00774_b200 as sdgp
    layer = inputs.ConvLayer("t", 3, 16, 16, 64, 128, 3, 3, 1, 1)
    dO, W = inputs.conv_layer_tensors(layer, seed=77)
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    for n, scheme in ((2, oracle.MAGNITUDE), (1, oracle.RANDOM), (2, oracle.RESCALED)):
        sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, 1, 1, n, 32, scheme, seed=5, flags=sdgp.FLAG_FUSED)
        check_no_device_error()
        pruned = oracle.prune(dO.reshape(-1, 128), n, 32, scheme, 5, want=("dense",))["dense"].reshape(dO.shape)
        assert_close(to_f64(dD), *conv_ref(pruned, W, 16, 16, 1, 1))
    x = torch.zeros((64, 128), dtype=torch.int16, device="cuda")
    w = torch.zeros((128, 64), dtype=torch.int16, device="cuda")
    y = torch.zeros((64, 64), dtype=torch.int16, device="cuda")
    with pytest.raises(sdgp.SdgpError) as e:
        sdgp.sdgp_dgrad_linear(x, w, y, 2, 32, sdgp.MAGNITUDE, flags=sdgp.FLAG_FUSED)
    assert e.value.status == 2


def test_unsupported_requests_raise():
    import paper_2202_00774_b200 as sdgp
    dO = torch.zeros((2, 4, 4, 128), dtype=torch.int16, device="cuda")
    W = torch.zeros((128, 3, 3, 64), dtype=torch.int16, device="cuda")
    dD = torch.zeros((2, 8, 8, 64), dtype=torch.int16, device="cuda")
    with pytest.raises(sdgp.SdgpError) as e:
        sdgp.sdgp_dgrad_conv2d(dO, W, dD, 3, 1, 2, 4, sdgp.MAGNITUDE, flags=sdgp.FLAG_DENSE)   # stride 3
    assert e.value.status == 2


# ------------------------------------------------- full benchmark sizes, sampled outputs


def _sampled_conv_check(layer, seed, n, m, scheme, samples=600, fused=False):
    """Run the two-pass (or fused) path on the full layer; compare `samples` output pixels (plus the
    first and last pixels of the tensor) with the oracle, which prunes only the rows those pixels read."""
    import paper_2202_00774_b200 as sdgp
    dO, W = inputs.conv_layer_tensors(layer, seed)
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    if fused:
        sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, 1, layer.pad, n, m, scheme, seed=5, flags=sdgp.FLAG_FUSED)
    else:
        ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(layer.B, layer.H, layer.W, layer.Cin, layer.Cout, layer.R,
                                                         layer.S, 1, layer.pad), dtype=torch.uint8, device="cuda")
        sdgp.sdgp_dgrad_conv2d(dev16(dO), dev16(W), dD, 1, layer.pad, n, m, scheme, seed=5, workspace=ws)
    check_no_device_error()
    got_all = dD.cpu().numpy().view(np.uint16)
    assert not np.isnan(inputs.bf16_bits_to_f32(got_all)).any()   # every output was written
    rng = np.random.default_rng(seed)
    # sample whole images so that the random scheme's linear indices and all borders are covered
    imgs = np.unique(np.concatenate([[0, layer.B - 1], rng.integers(0, layer.B, 6)]))
    per_img = layer.H * layer.W
    pruned = np.zeros_like(dO)
    for b in imgs:
        rows = dO[b].reshape(-1, layer.Cout)
        if scheme == oracle.RANDOM:
            # keys depend on the element's linear index in the whole tensor: prune a slab that
            # starts at row 0 of the tensor up to this image (cheap enough for the sampled images)
            full = oracle.prune(dO[:b + 1].reshape(-1, layer.Cout), n, m, scheme, 5, want=("dense",))["dense"]
            pruned[b] = full[-rows.shape[0]:].reshape(dO[b].shape)
        else:
            pruned[b] = oracle.prune(rows, n, m, scheme, 5, want=("dense",))["dense"].reshape(dO[b].shape)
    idx = np.concatenate([b * per_img + rng.integers(0, per_img, samples // len(imgs)) for b in imgs])
    edge = min(64, per_img)   # first pixels of the first image, last pixels of the last one
    idx = np.unique(np.concatenate([idx, np.arange(0, edge), np.arange(layer.B * per_img - edge, layer.B * per_img)]))
    got = inputs.bf16_bits_to_f32(got_all.reshape(-1, layer.Cin)[idx]).astype(np.float64)
    assert_close(got, *conv_ref(pruned, W, layer.H, layer.W, 1, layer.pad, pixel_index=idx), what=layer.name)


@pytest.mark.parametrize("index", range(7))
def test_resnet9_full_size_layers_sampled(index):
    """The benchmark's own shapes (batch 512) in the launch configuration it times."""
    layer = inputs.resnet9_layers(512)[index]
    scheme = [oracle.MAGNITUDE, oracle.RESCALED, oracle.RANDOM][index % 3]
    _sampled_conv_check(layer, seed=index, n=2, m=4, scheme=scheme)


@pytest.mark.parametrize("index,scheme", [(0, oracle.RANDOM), (1, oracle.MAGNITUDE), (3, oracle.RESCALED), (4, oracle.MAGNITUDE),
                                          (6, oracle.MAGNITUDE)])
def test_resnet9_full_size_layers_fused_sampled(index, scheme):
    """bench.py --mode fused: the same shapes with the prune inside the data-gradient kernel."""
    layer = inputs.resnet9_layers(512)[index]
    _sampled_conv_check(layer, seed=10 + index, n=2, m=4, scheme=scheme, fused=True)


def _device_conv_tensors(layer, seed):
    """dO (ReLU-masked Laplace) and W (He-normal) drawn on the device: the full-size ResNet-50 tensors take
    too long to draw on the host. Returned as int16 views of bf16."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    shape = layer.dO_shape()
    u = torch.rand(shape, generator=g, device="cuda") - 0.5
    lap = -torch.sign(u) * torch.log1p(-2 * u.abs())
    lap[torch.rand(shape, generator=g, device="cuda") < 0.5] = 0.0
    dO = lap.to(torch.bfloat16).view(torch.int16)
    del u, lap
    std = (2.0 / (layer.R * layer.S * layer.Cin)) ** 0.5
    W = (torch.randn(layer.W_shape(), generator=g, device="cuda") * std).to(torch.bfloat16).view(torch.int16)
    return dO, W


R50_FULL = [l.name for l, _ in inputs.resnet50_layers(256)]   # every distinct bottleneck convolution (23 shapes)


@pytest.mark.parametrize("name", R50_FULL)
def test_resnet50_full_size_layers_sampled(name):
    """ResNet-50 bottleneck shapes at batch 256, as `bench.py --workload resnet50` launches them (two-pass, 2:4
    magnitude): whole sampled images (first, last, three random) go to the oracle, 600 of their output pixels are compared."""
    import paper_2202_00774_b200 as sdgp
    layer = dict((l.name, l) for l, _ in inputs.resnet50_layers(256))[name]
    dO, W = _device_conv_tensors(layer, seed=len(name))
    ws = torch.empty(sdgp.sdgp_workspace_size_conv2d(layer.B, layer.H, layer.W, layer.Cin, layer.Cout, layer.R, layer.S,
                                                     layer.stride, layer.pad), dtype=torch.uint8, device="cuda")
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_conv2d(dO, W, dD, layer.stride, layer.pad, 2, 4, sdgp.MAGNITUDE, workspace=ws)
    check_no_device_error()
    assert not bool(torch.isnan(dD.view(torch.bfloat16)).any())          # every output was written
    rng = np.random.default_rng(len(name))
    imgs = np.unique(np.concatenate([[0, layer.B - 1], rng.integers(0, layer.B, 3)]))
    sub = dO[torch.from_numpy(imgs).cuda()].cpu().numpy().view(np.uint16)           # [len(imgs), P, Q, Cout]
    Wh = W.cpu().numpy().view(np.uint16)
    Cpad = (layer.Cout + 31) // 32 * 32
    flat = np.zeros((sub.size // layer.Cout, Cpad), np.uint16)
    flat[:, :layer.Cout] = sub.reshape(-1, layer.Cout)
    pruned = oracle.prune(flat, 2, 4, oracle.MAGNITUDE, want=("dense",))["dense"][:, :layer.Cout]
    pruned = np.ascontiguousarray(pruned).reshape(sub.shape)
    per_img = layer.H * layer.W
    idx = np.unique(np.concatenate([k * per_img + rng.integers(0, per_img, 120) for k in range(len(imgs))] +
                                   [np.arange(0, min(40, per_img)), len(imgs) * per_img - 1 - np.arange(0, min(40, per_img))]))
    got = to_f64(dD[torch.from_numpy(imgs).cuda()]).reshape(-1, layer.Cin)[idx]
    assert_close(got, *conv_ref(pruned, Wh, layer.H, layer.W, layer.stride, layer.pad, pixel_index=idx), what=name)


@pytest.mark.parametrize("n,m,scheme", [(2, 4, oracle.MAGNITUDE), (1, 4, oracle.RESCALED), (2, 8, oracle.MAGNITUDE),
                                        (2, 16, oracle.RESCALED)])
def test_gemm_large_full_size_sampled_rows(n, m, scheme):
    """[16384 x 4096] . [4096 x 4096] in full on the GPU; 96 sampled rows against the oracle."""
    import paper_2202_00774_b200 as sdgp
    c = inputs.GEMM_LARGE
    dO, W = inputs.fc_tensors(c["rows"], c["K"], c["N"], c["seed"])
    ws = torch.empty(sdgp.sdgp_workspace_size_linear(c["rows"], c["K"], c["N"]), dtype=torch.uint8, device="cuda")
    dD = torch.full((c["rows"], c["N"]), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_linear(dev16(dO), dev16(W), dD, n, m, scheme, seed=9, workspace=ws)
    check_no_device_error()
    rng = np.random.default_rng(n * 10 + m)
    rows = np.unique(np.concatenate([[0, 127, 128, c["rows"] - 1], rng.integers(0, c["rows"], 92)]))
    pruned = oracle.prune(dO[rows], n, m, scheme, 9, want=("dense",))["dense"]   # magnitude schemes: row-local
    got = inputs.bf16_bits_to_f32(dD[torch.from_numpy(rows).cuda()].cpu().numpy().view(np.uint16)).astype(np.float64)
    assert_close(got, *linear_ref(pruned, W))


def test_bounded_wait_reports_timeout_and_context_survives():
    """A wait that nothing satisfies gives up after its limit; the host sees SDGP_ERR_TIMEOUT once,
    and the next kernels run normally."""
    import paper_2202_00774_b200 as sdgp
    assert sdgp.sdgp_last_device_error() == 0
    sdgp.sdgp_selftest_bounded_wait()
    assert sdgp.sdgp_last_device_error() == 6
    assert sdgp.sdgp_last_device_error() == 0
    dO, W = inputs.fc_tensors(128, 128, 64, seed=1)
    dD = torch.empty((128, 64), dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_linear(dev16(dO), dev16(W), dD, 4, 4, sdgp.MAGNITUDE, flags=sdgp.FLAG_DENSE)
    check_no_device_error()
    assert_close(to_f64(dD), *linear_ref(dO, W))
