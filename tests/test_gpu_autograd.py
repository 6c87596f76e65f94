"""The torch.autograd front end: the input gradient it returns is prune(dL/dO) contracted with W
(oracle), the weight gradient is the framework's own, from the unpruned dL/dO (Section 3.1)."""
import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def rel_fro(got, ref):
    return np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)


def bits_to_tensor(bits, dtype):
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()
    return t.view(dtype)


@pytest.mark.parametrize("dtype,odt", [(torch.bfloat16, oracle.BF16), (torch.float16, oracle.FP16)])
def test_linear_layer_backward(dtype, odt):
    from paper_2202_00774_b200 import autograd as sa
    import paper_2202_00774_b200 as sdgp
    rows, Cin, Cout = 200, 128, 256
    rng = np.random.default_rng(0)
    x = torch.from_numpy(rng.standard_normal((rows, Cin)).astype(np.float32)).cuda().to(dtype).requires_grad_()
    w = torch.from_numpy((rng.standard_normal((Cout, Cin)) / 16).astype(np.float32)).cuda().to(dtype).requires_grad_()
    g = torch.from_numpy(rng.standard_normal((rows, Cout)).astype(np.float32)).cuda().to(dtype)
    y = sa.sdgp_linear(x, w, 2, 4, sdgp.RESCALED_MAGNITUDE, 0)
    y.backward(g)
    assert sdgp.sdgp_last_device_error() == 0
    g_bits = g.view(torch.int16).cpu().numpy().view(np.uint16)
    w_bits = w.detach().view(torch.int16).cpu().numpy().view(np.uint16)
    pruned = oracle.prune(g_bits, 2, 4, oracle.RESCALED, 0, want=("dense",), dtype=odt)["dense"]
    want = oracle.dgrad_linear(pruned, w_bits, dtype=odt)
    assert rel_fro(x.grad.float().cpu().numpy().astype(np.float64), want) <= 5e-3
    # the weight gradient comes from the UNPRUNED dL/dO
    ref_w = (g.float().t() @ x.detach().float()).cpu().numpy()
    assert rel_fro(w.grad.float().cpu().numpy(), ref_w) <= 1e-2


def test_conv_layer_backward_channels_last():
    from paper_2202_00774_b200 import autograd as sa
    import paper_2202_00774_b200 as sdgp
    B, Cin, Cout, H = 4, 64, 128, 16
    rng = np.random.default_rng(1)
    x = torch.from_numpy(rng.standard_normal((B, Cin, H, H)).astype(np.float32)).cuda().to(torch.bfloat16)
    x = x.contiguous(memory_format=torch.channels_last).requires_grad_()
    w = torch.from_numpy((rng.standard_normal((Cout, Cin, 3, 3)) / 24).astype(np.float32)).cuda().to(torch.bfloat16)
    w = w.contiguous(memory_format=torch.channels_last).requires_grad_()
    y = sa.sdgp_conv2d(x, w, 1, 1, 2, 4, sdgp.MAGNITUDE, 0)
    g = torch.from_numpy(rng.standard_normal(tuple(y.shape)).astype(np.float32)).cuda().to(torch.bfloat16)
    g = g.contiguous(memory_format=torch.channels_last)
    y.backward(g)
    assert sdgp.sdgp_last_device_error() == 0
    g_nhwc = g.permute(0, 2, 3, 1).contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    w_krsc = w.detach().permute(0, 2, 3, 1).contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    pruned = oracle.prune(g_nhwc.reshape(-1, Cout), 2, 4, oracle.MAGNITUDE, want=("dense",))["dense"].reshape(g_nhwc.shape)
    want = oracle.dgrad_conv2d(pruned, w_krsc, H, H, 1, 1)                     # NHWC
    got = x.grad.permute(0, 2, 3, 1).float().cpu().numpy().astype(np.float64)
    assert rel_fro(got, want) <= 5e-3
    ref_w = torch.nn.grad.conv2d_weight(x.detach().float(), w.shape, g.float(), 1, 1).cpu().numpy()
    assert rel_fro(w.grad.float().cpu().numpy(), ref_w) <= 1e-2


@pytest.mark.parametrize("pool", [False, True])
@pytest.mark.parametrize("Cout,n,m", [(128, 2, 4), (64, 2, 4), (128, 4, 8)])
def test_conv_relu_layer_backward_uses_the_producer(pool, Cout, n, m):
    """relu(conv2d) [+ max pooling]: dL/dO is formed and pruned by the producer; input gradient against the oracle's
    producer + contraction, weight gradient against the framework's own from the unpruned dL/dO."""
    from paper_2202_00774_b200 import autograd as sa
    import paper_2202_00774_b200 as sdgp
    B, Cin, H = 4, 64, 16
    rng = np.random.default_rng(2)
    x = torch.from_numpy(rng.standard_normal((B, Cin, H, H)).astype(np.float32)).cuda().to(torch.bfloat16)
    x = x.contiguous(memory_format=torch.channels_last).requires_grad_()
    w = torch.from_numpy((rng.standard_normal((Cout, Cin, 3, 3)) / 24).astype(np.float32)).cuda().to(torch.bfloat16)
    w = w.contiguous(memory_format=torch.channels_last).requires_grad_()
    y = sa.sdgp_conv2d_relu(x, w, 1, 1, pool, n, m, sdgp.MAGNITUDE, 0)
    with torch.no_grad():
        act = torch.relu(torch.nn.functional.conv2d(x, w, None, 1, 1))
        assert torch.equal(y, torch.nn.functional.max_pool2d(act, 2) if pool else act)
    g = torch.from_numpy(rng.standard_normal(tuple(y.shape)).astype(np.float32)).cuda().to(torch.bfloat16)
    g = g.contiguous(memory_format=torch.channels_last)
    y.backward(g)
    assert sdgp.sdgp_last_device_error() == 0
    nhwc = lambda t: t.permute(0, 2, 3, 1).contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    g_bits, a_bits = nhwc(g), nhwc(act)
    w_krsc = w.detach().permute(0, 2, 3, 1).contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    if pool:
        ref = oracle.maxpool_relu_backward_prune(g_bits, a_bits, n, m, oracle.MAGNITUDE, want=("dense",))
    else:
        ref = oracle.relu_backward_prune(g_bits.reshape(-1, Cout), a_bits.reshape(-1, Cout), n, m, oracle.MAGNITUDE, want=("dense",))
    want = oracle.dgrad_conv2d(ref["dense"].reshape(B, H, H, Cout), w_krsc, H, H, 1, 1)
    got = x.grad.permute(0, 2, 3, 1).float().cpu().numpy().astype(np.float64)
    assert rel_fro(got, want) <= 5e-3
    dO = torch.from_numpy(inputs.bf16_bits_to_f32(ref["grad"].reshape(B, H, H, Cout))).cuda().permute(0, 3, 1, 2)
    ref_w = torch.nn.grad.conv2d_weight(x.detach().float(), w.shape, dO.contiguous(), 1, 1).cpu().numpy()
    assert rel_fro(w.grad.float().cpu().numpy(), ref_w) <= 1e-2
