"""Data gradient of grouped convolutions and of channel counts that are not multiples of 64 (the RegNetX-400MF
shape set, Section 4) on the GPU vs the fp64 CPU oracle, through the C ABI. Tolerances as in test_gpu_dgrad.py:
relative Frobenius error <= 5e-3 and, per element, 2^-7 |ref| + 2^-16 sum |a||b|."""
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


def magnitudes(bits):
    return (np.asarray(bits).view(np.uint16) & np.uint16(0x7FFF)).astype(np.uint16)


def check(got, src, W, layer, what):
    ref = oracle.dgrad_conv2d_grouped(src, W, layer.H, layer.W, layer.groups, layer.stride, layer.pad)
    absdot = oracle.dgrad_conv2d_grouped(magnitudes(src), magnitudes(W), layer.H, layer.W, layer.groups, layer.stride, layer.pad)
    assert np.linalg.norm(got - ref) <= TOL * max(np.linalg.norm(ref), 1e-30), what
    bad = np.abs(got - ref) > 2.0 ** -7 * np.abs(ref) + 2.0 ** -16 * absdot
    assert not bad.any(), "%s: %d elements off, first at %s" % (what, int(bad.sum()), np.argwhere(bad)[0])


def run(layer, n, m, scheme, flags, seed=9):
    import paper_2202_00774_b200 as sdgp
    dO, W = inputs.conv_layer_tensors(layer, seed=seed)
    size = sdgp.sdgp_workspace_size_conv2d_grouped(layer.B, layer.H, layer.W, layer.Cin, layer.Cout, layer.R, layer.S,
                                                   layer.stride, layer.pad, layer.groups, flags)
    ws = torch.empty(size, dtype=torch.uint8, device="cuda")
    dD = torch.full(layer.dD_shape(), -1, dtype=torch.int16, device="cuda")
    sdgp.sdgp_dgrad_conv2d_grouped(dev16(dO), dev16(W), dD, layer.stride, layer.pad, layer.groups, n, m, scheme, seed=77,
                                   workspace=ws, flags=flags)
    assert sdgp.sdgp_last_device_error() == 0
    if flags == sdgp.FLAG_DENSE or n == m:
        src = dO
    else:
        src = oracle.prune(dO.reshape(-1, layer.Cout), n, m, scheme, 77, want=("dense",))["dense"].reshape(dO.shape)
    check(to_f64(dD), src, W, layer, "%s flags=%d %d:%d" % (layer.name, flags, n, m))


REGNETX = {l.name: l for l in inputs.regnetx_400mf_layers(batch=3)}


@pytest.mark.parametrize("name", sorted(REGNETX))
@pytest.mark.parametrize("mode", ["two_pass", "dense"])
def test_regnetx_400mf_layers(name, mode):
    import paper_2202_00774_b200 as sdgp
    run(REGNETX[name], 2, 4, oracle.MAGNITUDE, sdgp.FLAG_TWO_PASS if mode == "two_pass" else sdgp.FLAG_DENSE)


GROUPED = [l for l in inputs.regnetx_400mf_layers(batch=2) if l.groups > 1]


@pytest.mark.parametrize("layer", GROUPED, ids=[l.name for l in GROUPED])
@pytest.mark.parametrize("n,m,scheme", [(1, 4, oracle.RESCALED), (2, 8, oracle.RANDOM), (2, 16, oracle.MAGNITUDE)])
def test_grouped_layers_other_patterns(layer, n, m, scheme):
    import paper_2202_00774_b200 as sdgp
    run(layer, n, m, scheme, sdgp.FLAG_TWO_PASS)


@pytest.mark.parametrize("layer", GROUPED, ids=[l.name for l in GROUPED])
def test_grouped_layers_masked(layer):
    import paper_2202_00774_b200 as sdgp
    run(layer, 4, 8, oracle.MAGNITUDE, sdgp.FLAG_MASKED)


@pytest.mark.parametrize("layer", [l for l in GROUPED if l.Cin % 64 == 0], ids=[l.name for l in GROUPED if l.Cin % 64 == 0])
def test_grouped_layers_fused(layer):
    import paper_2202_00774_b200 as sdgp
    run(layer, 2, 4, oracle.MAGNITUDE, sdgp.FLAG_FUSED)


def test_fused_refuses_padded_channel_counts():
    import paper_2202_00774_b200 as sdgp
    layer = inputs.ConvLayer("t", 1, 8, 8, 32, 32, 3, 3, 1, 1, 2)
    with pytest.raises(sdgp.SdgpError) as e:
        run(layer, 2, 4, oracle.MAGNITUDE, sdgp.FLAG_FUSED)
    assert e.value.status == 2      # SDGP_ERR_UNSUPPORTED


@pytest.mark.parametrize("B,H,Wd,Cin,Cout,R,S,stride,pad,groups", [
    (5, 14, 14, 160, 160, 3, 3, 1, 1, 10),     # several strips, ragged channel blocks on both sides
    (2, 28, 28, 96, 48, 3, 3, 2, 1, 3),        # 32 input and 16 output channels per group
    (4, 7, 7, 64, 128, 3, 3, 1, 1, 8),         # general kernel (7 x 7 images)
    (3, 16, 16, 40, 80, 1, 1, 1, 0, 1),        # no groups, channel counts that are multiples of 8 only
    (2, 12, 20, 128, 128, 3, 3, 1, 1, 1),      # groups == 1 with aligned channel counts: the ordinary path
])
def test_other_grouped_shapes(B, H, Wd, Cin, Cout, R, S, stride, pad, groups):
    import paper_2202_00774_b200 as sdgp
    layer = inputs.ConvLayer("case", B, H, Wd, Cin, Cout, R, S, stride, pad, groups)
    for flags in (sdgp.FLAG_TWO_PASS, sdgp.FLAG_DENSE):
        run(layer, 2, 4, oracle.MAGNITUDE, flags)


def test_argument_errors():
    import paper_2202_00774_b200 as sdgp
    layer = inputs.ConvLayer("t", 1, 8, 8, 32, 32, 3, 3, 1, 1, 2)
    dO, W = inputs.conv_layer_tensors(layer, seed=1)
    dD = torch.zeros(layer.dD_shape(), dtype=torch.int16, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(sdgp.SdgpError) as e:      # 3 groups do not divide 32 channels
        sdgp.sdgp_dgrad_conv2d_grouped(dev16(dO), dev16(W), dD, 1, 1, 3, 2, 4, sdgp.MAGNITUDE, workspace=ws)
    assert e.value.status == 1
    with pytest.raises(sdgp.SdgpError) as e:      # no workspace
        sdgp.sdgp_dgrad_conv2d_grouped(dev16(dO), dev16(W), dD, 1, 1, 2, 2, 4, sdgp.MAGNITUDE, workspace=None)
    assert e.value.status == 4
    with pytest.raises(sdgp.SdgpError) as e:      # 4 input channels per group: below one 16-byte vector
        sdgp.sdgp_dgrad_conv2d_grouped(dev16(dO), dev16(W[..., :4].copy()), dD, 1, 1, 8, 2, 4, sdgp.MAGNITUDE, workspace=ws)
    assert e.value.status == 2
