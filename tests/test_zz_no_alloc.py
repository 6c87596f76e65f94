"""sdgp_dgrad_linear_static - the entry point for callers that cannot allocate device memory
(its scratch is a fixed array inside the library) - must give what sdgp_dgrad_linear gives
with a caller-supplied workspace, bit for bit: both run the same two kernels on the same inputs.
Two calls in a row with different inputs share the array; the second must not see anything the
first left behind. Each result is also checked against the CPU oracle. Collected last on purpose."""
import numpy as np
import pytest

import oracle
from paper_2202_00774_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 5e-3


def _f64(t):
    return inputs.bf16_bits_to_f32(t.cpu().numpy().view(np.uint16)).astype(np.float64)


def _dev16(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()


def test_static_scratch_matches_workspace_variant_twice():
    import paper_2202_00774_b200 as sdgp
    # the second call is smaller in rows, larger in K: its rows lie over the first call's leftovers;
    # the third prunes nothing (n == m) and must leave the shared array alone
    calls = [(700, 512, 256, 2, 4, sdgp.MAGNITUDE, 11), (333, 1024, 128, 2, 8, sdgp.RESCALED_MAGNITUDE, 12),
             (200, 256, 64, 4, 4, sdgp.MAGNITUDE, 13)]
    for rows, K, N, n, m, scheme, seed in calls:
        dO, W = inputs.fc_tensors(rows, K, N, seed=seed)
        d_dO, d_W = _dev16(dO), _dev16(W)
        ws = torch.empty(sdgp.sdgp_workspace_size_linear(rows, K, N), dtype=torch.uint8, device="cuda")
        want = torch.full((rows, N), -1, dtype=torch.int16, device="cuda")
        got = torch.full((rows, N), -2, dtype=torch.int16, device="cuda")
        sdgp.sdgp_dgrad_linear(d_dO, d_W, want, n, m, scheme, seed=seed, workspace=ws)
        sdgp.sdgp_dgrad_linear_static(d_dO, d_W, got, n, m, scheme, seed=seed)
        torch.cuda.synchronize()
        assert sdgp.sdgp_last_device_error() == 0
        assert torch.equal(got, want)          # same kernels, same inputs: identical bits
        pruned = oracle.prune(dO, n, m, scheme, seed, want=("dense",))["dense"]
        ref = oracle.dgrad_linear(pruned, W)
        assert np.linalg.norm(_f64(got) - ref) <= TOL * np.linalg.norm(ref)


def test_static_scratch_rejects_oversized_problems():
    import paper_2202_00774_b200 as sdgp
    rows, K, N = 8193, 1024, 64  # rows*K just above the 8Mi-element limit; nothing is launched
    x = torch.zeros((rows, K), dtype=torch.int16, device="cuda")
    w = torch.zeros((K, N), dtype=torch.int16, device="cuda")
    y = torch.zeros((rows, N), dtype=torch.int16, device="cuda")
    with pytest.raises(sdgp.SdgpError) as e:
        sdgp.sdgp_dgrad_linear_static(x, w, y, 2, 4, sdgp.MAGNITUDE)
    assert e.value.status == 7
    assert "scratch" in sdgp.status_string(7)
