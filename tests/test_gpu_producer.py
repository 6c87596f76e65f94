"""sdgp_relu_backward_prune on the GPU against the oracle's producer (ReLU backward, then Algorithm 1): every output
bit for bit, and the sparse contraction fed from it within the data-gradient tolerance."""
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


def make(rows, K, seed, dtype=oracle.BF16):
    rng = np.random.default_rng(seed)
    to_bits = inputs.f32_to_bf16_bits if dtype == oracle.BF16 else (lambda x: x.astype(np.float16).view(np.uint16))
    dY = to_bits(rng.laplace(size=(rows, K)).astype(np.float32))
    act = to_bits(np.maximum(rng.standard_normal((rows, K)), 0.0).astype(np.float32))
    # a few special activations: -0.0, NaN, +Inf, the smallest subnormal, a negative number
    flat = act.reshape(-1)
    special = [0x8000, 0x7FC0 if dtype == oracle.BF16 else 0x7E00, 0x7F80 if dtype == oracle.BF16 else 0x7C00, 0x0001, 0xBF80]
    flat[rng.integers(0, flat.size, 400)] = np.resize(np.array(special, np.uint16), 400)
    return dY, act


@pytest.mark.parametrize("n,m", [(2, 4), (1, 4), (2, 8), (1, 8), (2, 16), (2, 32)])
@pytest.mark.parametrize("scheme", [oracle.MAGNITUDE, oracle.RESCALED, oracle.RANDOM])
def test_producer_outputs_bit_exact(n, m, scheme):
    import paper_2202_00774_b200 as sdgp
    rows, K = 1237, 160                 # ragged: not a whole number of thread blocks
    dY, act = make(rows, K, seed=n * 10 + m)
    grad = torch.full((rows, K), -1, dtype=torch.int16, device="cuda")
    dense = torch.full((rows, K), -1, dtype=torch.int16, device="cuda")
    values = torch.full((rows, K // 2), -1, dtype=torch.int16, device="cuda")
    meta = torch.full((rows, K // 16), -1, dtype=torch.int16, device="cuda")
    mask = torch.full((rows, K // 32), -1, dtype=torch.int32, device="cuda")
    sdgp.sdgp_relu_backward_prune(dev16(dY), dev16(act), n, m, scheme, seed=77, grad=grad, dense=dense, values=values,
                                  meta=meta, mask=mask)
    ref = oracle.relu_backward_prune(dY, act, n, m, scheme, seed=77)
    assert np.array_equal(host16(grad), ref["grad"])
    assert np.array_equal(host16(dense), ref["dense"])
    assert np.array_equal(host16(values), ref["values"])
    assert np.array_equal(host16(meta), ref["meta"])
    assert np.array_equal(mask.cpu().numpy().view(np.uint32), ref["mask"])


def test_producer_binary16_and_plain_relu_backward():
    import paper_2202_00774_b200 as sdgp
    rows, K = 515, 128
    dY, act = make(rows, K, seed=3, dtype=oracle.FP16)
    grad = torch.full((rows, K), -1, dtype=torch.int16, device="cuda")
    values = torch.full((rows, K // 2), -1, dtype=torch.int16, device="cuda")
    meta = torch.full((rows, K // 16), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_relu_backward_prune(dev16(dY), dev16(act), 2, 4, sdgp.RESCALED_MAGNITUDE, seed=1, dtype=sdgp.FP16, grad=grad,
                                  values=values, meta=meta)
    ref = oracle.relu_backward_prune(dY, act, 2, 4, oracle.RESCALED, seed=1, dtype=oracle.FP16)
    assert np.array_equal(host16(grad), ref["grad"])
    assert np.array_equal(host16(values), ref["values"])
    assert np.array_equal(host16(meta), ref["meta"])
    # n == m: nothing pruned, the call is the ReLU backward alone
    grad.fill_(-1)
    sdgp.sdgp_relu_backward_prune(dev16(dY), dev16(act), 4, 4, sdgp.MAGNITUDE, dtype=sdgp.FP16, grad=grad)
    assert np.array_equal(host16(grad), oracle.relu_backward(dY, act, oracle.FP16))


def test_producer_feeds_the_sparse_contraction():
    """ReLU backward + prune in one pass, then the contraction alone: a 1 x 1 convolution of ResNet-50's shape family."""
    import paper_2202_00774_b200 as sdgp
    B, HW, Cin, Cout = 4, 14, 256, 1024
    rows = B * HW * HW
    dY, act = make(rows, Cout, seed=8)
    W = inputs.f32_to_bf16_bits((np.random.default_rng(1).standard_normal((Cout, Cin)) * (2.0 / Cin) ** 0.5).astype(np.float32))
    values = torch.empty((rows, Cout // 2), dtype=torch.int16, device="cuda")
    meta = torch.empty((rows, Cout // 16), dtype=torch.int16, device="cuda")
    dD = torch.full((B, HW, HW, Cin), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_relu_backward_prune(dev16(dY), dev16(act), 2, 4, sdgp.MAGNITUDE, values=values, meta=meta)
    sdgp.sdgp_spmm_conv2d(values.view(B, HW, HW, Cout // 2), meta.view(B, HW, HW, Cout // 16), dev16(W).view(Cout, 1, 1, Cin), dD, 1, 0)
    assert sdgp.sdgp_last_device_error() == 0
    ref = oracle.relu_backward_prune(dY, act, 2, 4, oracle.MAGNITUDE, want=("dense",))
    want = oracle.dgrad_linear(ref["dense"], W)
    got = inputs.bf16_bits_to_f32(host16(dD)).astype(np.float64).reshape(rows, Cin)
    assert np.linalg.norm(got - want) <= TOL * np.linalg.norm(want)


def test_producer_rejects_bad_arguments():
    import paper_2202_00774_b200 as sdgp
    x = torch.zeros((8, 64), dtype=torch.int16, device="cuda")
    v = torch.zeros((8, 32), dtype=torch.int16, device="cuda")
    with pytest.raises(sdgp.SdgpError) as e:
        sdgp.sdgp_relu_backward_prune(x, x, 4, 8, sdgp.MAGNITUDE, values=v)      # 4:8 has no compressed form
    assert e.value.status == 2
    with pytest.raises(sdgp.SdgpError) as e:
        sdgp.sdgp_relu_backward_prune(x, x, 0, 4, sdgp.MAGNITUDE, grad=x)
    assert e.value.status == 1


# ---- the producer below the ReLU that follows a residual addition: two gradients are added before the gate ----


def make_skip(rows, K, seed, dtype=oracle.BF16):
    """A second gradient with the cases of the addition that matter: a different scale (operands that half-vanish), exact
    negatives of dY (cancellation to +0.0), zeros of both signs, infinities of both signs and NaNs."""
    rng = np.random.default_rng(seed + 1000)
    to_bits = inputs.f32_to_bf16_bits if dtype == oracle.BF16 else (lambda x: x.astype(np.float16).view(np.uint16))
    scale = np.exp2(rng.integers(-12, 4, size=(rows, K))).astype(np.float32)
    dSkip = to_bits((rng.laplace(size=(rows, K)) * scale).astype(np.float32))
    return dSkip


@pytest.mark.parametrize("n,m,scheme", [(2, 4, oracle.MAGNITUDE), (2, 4, oracle.RESCALED), (1, 4, oracle.RANDOM),
                                        (2, 8, oracle.MAGNITUDE), (2, 16, oracle.RESCALED), (2, 32, oracle.RANDOM)])
@pytest.mark.parametrize("dtype", [oracle.BF16, oracle.FP16])
def test_residual_producer_outputs_bit_exact(n, m, scheme, dtype):
    import paper_2202_00774_b200 as sdgp
    rows, K = 1237, 160
    dY, act = make(rows, K, seed=n * 10 + m, dtype=dtype)
    dSkip = make_skip(rows, K, seed=n * 10 + m, dtype=dtype)
    inf, nan = (0x7F80, 0x7FC1) if dtype == oracle.BF16 else (0x7C00, 0x7E01)
    fy, fs = dY.reshape(-1), dSkip.reshape(-1)
    fs[0:4000:7] = fy[0:4000:7] ^ 0x8000                      # x + (-x)
    fy[1:3000:11], fs[1:3000:11] = 0x8000, 0x0000             # -0 + +0
    fy[2:3000:13], fs[2:3000:13] = 0x8000, 0x8000             # -0 + -0 (stays -0.0 where the ReLU passes it)
    fy[3:3000:17], fs[3:3000:17] = inf, inf | 0x8000          # inf - inf: the canonical NaN
    fy[4:3000:19] = nan                                       # a NaN with a payload: canonical after the addition
    fy[5:3000:23], fs[5:3000:23] = inf - 1, inf - 1           # the largest finite number twice: overflow to infinity
    dt = sdgp.BF16 if dtype == oracle.BF16 else sdgp.FP16
    grad = torch.full((rows, K), -1, dtype=torch.int16, device="cuda")
    dense = torch.full((rows, K), -1, dtype=torch.int16, device="cuda")
    values = torch.full((rows, K // 2), -1, dtype=torch.int16, device="cuda")
    meta = torch.full((rows, K // 16), -1, dtype=torch.int16, device="cuda")
    mask = torch.full((rows, K // 32), -1, dtype=torch.int32, device="cuda")
    d_dY, d_skip, d_act = dev16(dY), dev16(dSkip), dev16(act)
    sdgp.sdgp_residual_relu_backward_prune(d_dY, d_skip, d_act, n, m, scheme, seed=77, dtype=dt, grad=grad, dense=dense,
                                           values=values, meta=meta, mask=mask)
    ref = oracle.residual_relu_backward_prune(dY, dSkip, act, n, m, scheme, seed=77, dtype=dtype)
    assert np.array_equal(host16(grad), ref["grad"])
    assert np.array_equal(host16(dense), ref["dense"])
    assert np.array_equal(host16(values), ref["values"])
    assert np.array_equal(host16(meta), ref["meta"])
    assert np.array_equal(mask.cpu().numpy().view(np.uint32), ref["mask"])
    # the inputs are never written
    assert np.array_equal(host16(d_dY), dY) and np.array_equal(host16(d_skip), dSkip) and np.array_equal(host16(d_act), act)


def test_residual_producer_plain_sum_and_the_sparse_contraction():
    import paper_2202_00774_b200 as sdgp
    B, HW, Cin, Cout = 4, 14, 128, 512
    rows = B * HW * HW
    dY, act = make(rows, Cout, seed=21)
    dSkip = make_skip(rows, Cout, seed=21)
    # n == m: the gated sum alone (what the weight gradient reads)
    grad = torch.full((rows, Cout), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_residual_relu_backward_prune(dev16(dY), dev16(dSkip), dev16(act), 4, 4, sdgp.MAGNITUDE, grad=grad)
    assert np.array_equal(host16(grad), oracle.residual_relu_backward(dY, dSkip, act))
    # compressed outputs straight into the contraction
    W = inputs.f32_to_bf16_bits((np.random.default_rng(2).standard_normal((Cout, Cin)) * (2.0 / Cin) ** 0.5).astype(np.float32))
    values = torch.empty((rows, Cout // 2), dtype=torch.int16, device="cuda")
    meta = torch.empty((rows, Cout // 16), dtype=torch.int16, device="cuda")
    dD = torch.full((B, HW, HW, Cin), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_residual_relu_backward_prune(dev16(dY), dev16(dSkip), dev16(act), 2, 4, sdgp.MAGNITUDE, values=values, meta=meta)
    sdgp.sdgp_spmm_conv2d(values.view(B, HW, HW, Cout // 2), meta.view(B, HW, HW, Cout // 16), dev16(W).view(Cout, 1, 1, Cin), dD, 1, 0)
    assert sdgp.sdgp_last_device_error() == 0
    ref = oracle.residual_relu_backward_prune(dY, dSkip, act, 2, 4, oracle.MAGNITUDE, want=("dense",))
    want = oracle.dgrad_linear(ref["dense"], W)
    got = inputs.bf16_bits_to_f32(host16(dD)).astype(np.float64).reshape(rows, Cin)
    assert np.linalg.norm(got - want) <= TOL * np.linalg.norm(want)


def test_residual_producer_rejects_bad_arguments():
    import paper_2202_00774_b200 as sdgp
    x = torch.zeros((8, 64), dtype=torch.int16, device="cuda")
    with pytest.raises(sdgp.SdgpError) as e:
        sdgp.sdgp_residual_relu_backward_prune(x, None, x, 2, 4, sdgp.MAGNITUDE, grad=x)
    assert e.value.status == 1
    with pytest.raises(sdgp.SdgpError) as e:
        odd = torch.zeros(8 * 64 + 8, dtype=torch.int16, device="cuda")[1:1 + 8 * 64].view(8, 64)   # 2 bytes off a 16-byte boundary
        sdgp.sdgp_residual_relu_backward_prune(x, odd, x, 2, 4, sdgp.MAGNITUDE, grad=torch.zeros_like(x))
    assert e.value.status == 3


# ---- the producer below a ReLU followed by 2 x 2 max pooling: the pooled gradient goes to each window's maximum ----


def make_pool(B, H, W, K, seed, dtype=oracle.BF16, nan_gradients=True):
    rng = np.random.default_rng(seed + 2000)
    to_bits = inputs.f32_to_bf16_bits if dtype == oracle.BF16 else (lambda x: x.astype(np.float16).view(np.uint16))
    # coarse activations: equal values inside a window are common; all-negative windows occur too
    act = to_bits((np.round(rng.standard_normal((B, H, W, K)) * 2.0) / 2.0).astype(np.float32))
    flat = act.reshape(-1)
    special = [0x8000, 0x7FC0 if dtype == oracle.BF16 else 0x7E00, 0x7F80 if dtype == oracle.BF16 else 0x7C00, 0x0001, 0xBF80]
    flat[rng.integers(0, flat.size, 600)] = np.resize(np.array(special, np.uint16), 600)
    g = to_bits(rng.laplace(size=(B, H // 2, W // 2, K)).astype(np.float32))
    if nan_gradients:
        g.reshape(-1)[rng.integers(0, g.size, 50)] = 0x7FC1   # payloads travel unchanged
    return g, act


@pytest.mark.parametrize("n,m,scheme", [(2, 4, oracle.MAGNITUDE), (2, 4, oracle.RESCALED), (1, 4, oracle.RANDOM),
                                        (3, 4, oracle.MAGNITUDE), (2, 8, oracle.MAGNITUDE), (2, 16, oracle.RESCALED),
                                        (2, 32, oracle.RANDOM)])
@pytest.mark.parametrize("shape", [(3, 6, 10, 160), (5, 2, 2, 32), (2, 16, 16, 128)])
def test_maxpool_producer_outputs_bit_exact(n, m, scheme, shape):
    import paper_2202_00774_b200 as sdgp
    B, H, W, K = shape
    if K % m:
        pytest.skip("K is not a multiple of m")
    g, act = make_pool(B, H, W, K, seed=n * 10 + m)
    rows = B * H * W
    compressed = n <= 2
    grad = torch.full((B, H, W, K), -1, dtype=torch.int16, device="cuda")
    dense = torch.full((rows, K), -1, dtype=torch.int16, device="cuda")
    values = torch.full((rows, K // 2), -1, dtype=torch.int16, device="cuda") if compressed else None
    meta = torch.full((rows, K // 16), -1, dtype=torch.int16, device="cuda") if compressed else None
    mask = torch.full((rows, K // 32), -1, dtype=torch.int32, device="cuda")
    d_g, d_act = dev16(g), dev16(act)
    sdgp.sdgp_maxpool_relu_backward_prune(d_g, d_act, n, m, scheme, seed=99, grad=grad, dense=dense, values=values, meta=meta,
                                          mask=mask)
    want = ("dense", "values", "meta", "mask") if compressed else ("dense", "mask")
    ref = oracle.maxpool_relu_backward_prune(g, act, n, m, scheme, seed=99, want=want)
    assert np.array_equal(host16(grad), ref["grad"])
    assert np.array_equal(host16(dense), ref["dense"])
    if compressed:
        assert np.array_equal(host16(values), ref["values"])
        assert np.array_equal(host16(meta), ref["meta"])
    assert np.array_equal(mask.cpu().numpy().view(np.uint32), ref["mask"])
    assert np.array_equal(host16(d_g), g) and np.array_equal(host16(d_act), act)


def test_maxpool_producer_binary16_plain_backward_and_the_sparse_contraction():
    import paper_2202_00774_b200 as sdgp
    B, H, W, Cin, Cout = 4, 8, 8, 64, 128
    g, act = make_pool(B, H, W, Cout, seed=5, dtype=oracle.FP16)
    grad = torch.full((B, H, W, Cout), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_maxpool_relu_backward_prune(dev16(g), dev16(act), 4, 4, sdgp.MAGNITUDE, dtype=sdgp.FP16, grad=grad)   # n == m: no pruning
    assert np.array_equal(host16(grad), oracle.maxpool_relu_backward(g, act, oracle.FP16))
    # bf16, compressed outputs straight into a 3 x 3 convolution's contraction
    g, act = make_pool(B, H, W, Cout, seed=6, nan_gradients=False)
    layer = inputs.ConvLayer("pool", B, H, W, Cin, Cout, 3, 3, 1, 1)
    _, Wt = inputs.conv_layer_tensors(layer, seed=3)
    rows = B * H * W
    values = torch.empty((rows, Cout // 2), dtype=torch.int16, device="cuda")
    meta = torch.empty((rows, Cout // 16), dtype=torch.int16, device="cuda")
    dD = torch.full((B, H, W, Cin), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_maxpool_relu_backward_prune(dev16(g), dev16(act), 2, 4, sdgp.MAGNITUDE, values=values, meta=meta)
    sdgp.sdgp_spmm_conv2d(values.view(B, H, W, Cout // 2), meta.view(B, H, W, Cout // 16), dev16(Wt), dD, 1, 1)
    assert sdgp.sdgp_last_device_error() == 0
    ref = oracle.maxpool_relu_backward_prune(g, act, 2, 4, oracle.MAGNITUDE, want=("dense",))
    pruned = ref["dense"].reshape(B, H, W, Cout)
    want = oracle.dgrad_conv2d(pruned, Wt, H, W, 1, 1)
    got = inputs.bf16_bits_to_f32(host16(dD)).astype(np.float64)
    assert np.linalg.norm(got - want) <= TOL * np.linalg.norm(want)


def test_maxpool_producer_rejects_bad_arguments():
    import paper_2202_00774_b200 as sdgp
    act = torch.zeros((2, 3, 4, 64), dtype=torch.int16, device="cuda")      # odd height
    g = torch.zeros((2, 1, 2, 64), dtype=torch.int16, device="cuda")
    with pytest.raises(sdgp.SdgpError) as e:
        sdgp.sdgp_maxpool_relu_backward_prune(g, act, 2, 4, sdgp.MAGNITUDE, grad=act)
    assert e.value.status == 1
    act = torch.zeros((2, 4, 4, 64), dtype=torch.int16, device="cuda")
    g = torch.zeros((2, 2, 2, 64), dtype=torch.int16, device="cuda")
    with pytest.raises(sdgp.SdgpError) as e:
        sdgp.sdgp_maxpool_relu_backward_prune(g, act, 4, 8, sdgp.MAGNITUDE, grad=act)     # groups of 8 keep one or two
    assert e.value.status == 2
    with pytest.raises(ValueError):
        sdgp.sdgp_maxpool_relu_backward_prune(act, act, 2, 4, sdgp.MAGNITUDE, grad=act)   # gradient not of the pooled shape


@pytest.mark.parametrize("dtype", [oracle.BF16, oracle.FP16])
def test_maxpool_producer_with_a_second_pooled_gradient(dtype):
    """ResNet-9: a residual block follows the pooling, so the pooling's output receives two gradients."""
    import paper_2202_00774_b200 as sdgp
    B, H, W, K = 3, 8, 6, 128
    g, act = make_pool(B, H, W, K, seed=31, dtype=dtype)
    skip = make_skip(B * (H // 2) * (W // 2), K, seed=31, dtype=dtype).reshape(g.shape)
    skip.reshape(-1)[0:500:3] = g.reshape(-1)[0:500:3] ^ 0x8000           # cancellations
    dt = sdgp.BF16 if dtype == oracle.BF16 else sdgp.FP16
    rows = B * H * W
    grad = torch.full((B, H, W, K), -1, dtype=torch.int16, device="cuda")
    values = torch.full((rows, K // 2), -1, dtype=torch.int16, device="cuda")
    meta = torch.full((rows, K // 16), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_maxpool_relu_backward_prune(dev16(g), dev16(act), 2, 8, sdgp.RESCALED_MAGNITUDE, seed=5, dtype=dt, grad=grad,
                                          values=values, meta=meta, skip=dev16(skip))
    ref = oracle.maxpool_relu_backward_prune(g, act, 2, 8, oracle.RESCALED, seed=5, want=("values", "meta"), dtype=dtype, skip=skip)
    assert np.array_equal(host16(grad), ref["grad"])
    assert np.array_equal(host16(values), ref["values"])
    assert np.array_equal(host16(meta), ref["meta"])
