"""Host-only checks of the C-ABI library: it loads without a GPU, exports every symbol the
header declares, and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2202_00774_b200 import binding
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sdgp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sdgp_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert "sdgp_prune" in names and "sdgp_dgrad_linear" in names and "sdgp_dgrad_conv2d" in names
    for name in names:
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols():
    from paper_2202_00774_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()


def test_status_strings(lib):
    seen = {lib.sdgp_status_string(i).decode() for i in range(8)}
    assert len(seen) == 8 and "ok" in seen and "unknown status" not in seen
    assert lib.sdgp_status_string(99).decode() == "unknown status"


FAKE = ctypes.c_void_p(0x1000)  # aligned, never dereferenced: every call below fails validation first


def test_prune_rejects_bad_arguments_before_launch(lib):
    P = lib.sdgp_prune
    assert P(FAKE, 4, 64, 2, 4, 1, 0, None, None, None, None, None) in (0, 5)  # valid args: OK, or CUDA error with no GPU
    assert P(FAKE, 4, 64, 0, 4, 1, 0, FAKE, None, None, None, None) == 1   # n < 1
    assert P(FAKE, 4, 64, 5, 4, 1, 0, FAKE, None, None, None, None) == 1   # n > m
    assert P(FAKE, 4, 64, 2, 64, 1, 0, FAKE, None, None, None, None) == 1  # m > 32
    assert P(FAKE, 4, 64, 2, 6, 1, 0, FAKE, None, None, None, None) == 2   # m not a supported group size
    assert P(FAKE, 4, 72, 2, 16, 1, 0, FAKE, None, None, None, None) == 1  # K % m != 0
    assert P(FAKE, 4, 64, 2, 4, 7, 0, FAKE, None, None, None, None) == 1   # unknown scheme
    assert P(FAKE, -1, 64, 2, 4, 1, 0, FAKE, None, None, None, None) == 1
    assert P(None, 4, 64, 2, 4, 1, 0, FAKE, None, None, None, None) == 1   # null input
    assert P(FAKE, 4, 64, 4, 8, 1, 0, None, FAKE, FAKE, None, None) == 2   # 4:8 has no compressed form
    assert P(FAKE, 4, 40, 2, 4, 1, 0, FAKE, None, None, None, None) == 3   # K % 16 != 0
    assert P(FAKE, 4, 48, 2, 4, 1, 0, None, None, None, FAKE, None) == 3   # mask needs K % 32 == 0
    assert P(ctypes.c_void_p(0x1008), 4, 64, 2, 4, 1, 0, FAKE, None, None, None, None) == 3
    assert P(None, 0, 64, 2, 4, 1, 0, None, None, None, None, None) == 0   # empty tensor: no-op


def test_producers_reject_bad_arguments_before_launch(lib):
    i64, i32, u64, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_uint64, ctypes.c_void_p
    Pr, Rs = lib.sdgp_relu_backward_prune, lib.sdgp_residual_relu_backward_prune
    Pr.argtypes = [vp, vp, i64, i64, i32, i32, i32, u64, i32, vp, vp, vp, vp, vp, vp]
    Rs.argtypes = [vp, vp, vp, i64, i64, i32, i32, i32, u64, i32, vp, vp, vp, vp, vp, vp]
    assert Pr(FAKE, None, 4, 64, 2, 4, 1, 0, 0, FAKE, None, None, None, None, None) == 1       # no activation
    assert Rs(FAKE, None, FAKE, 4, 64, 2, 4, 1, 0, 0, FAKE, None, None, None, None, None) == 1  # no second gradient
    assert Rs(FAKE, FAKE, None, 4, 64, 2, 4, 1, 0, 0, FAKE, None, None, None, None, None) == 1
    assert Rs(FAKE, ctypes.c_void_p(0x1002), FAKE, 4, 64, 2, 4, 1, 0, 0, FAKE, None, None, None, None, None) == 3
    assert Rs(FAKE, FAKE, FAKE, 4, 64, 4, 8, 1, 0, 0, None, None, FAKE, FAKE, None, None) == 2   # 4:8 has no compressed form
    assert Rs(FAKE, FAKE, FAKE, 4, 64, 2, 4, 1, 0, 9, FAKE, None, None, None, None, None) == 1   # unknown element type
    assert Rs(None, None, None, 0, 64, 2, 4, 1, 0, 0, None, None, None, None, None, None) == 0   # empty tensor: no-op
    Mp = lib.sdgp_maxpool_relu_backward_prune
    Mp.argtypes = [vp, vp, vp, i32, i32, i32, i64, i32, i32, i32, u64, i32, vp, vp, vp, vp, vp, vp]
    assert Mp(FAKE, None, FAKE, 2, 3, 4, 64, 2, 4, 1, 0, 0, FAKE, None, None, None, None, None) == 1    # odd height
    assert Mp(FAKE, None, FAKE, 2, 4, 6, 72, 2, 16, 1, 0, 0, FAKE, None, None, None, None, None) == 1   # K % m != 0
    assert Mp(FAKE, None, None, 2, 4, 4, 64, 2, 4, 1, 0, 0, FAKE, None, None, None, None, None) == 1    # no activation
    assert Mp(FAKE, FAKE, FAKE, 2, 4, 4, 64, 4, 8, 1, 0, 0, FAKE, None, None, None, None, None) == 2
    assert Mp(FAKE, None, FAKE, 2, 4, 4, 40, 2, 4, 1, 0, 0, FAKE, None, None, None, None, None) == 3    # K % 16 != 0
    assert Mp(FAKE, None, FAKE, 1 << 20, 1 << 10, 1 << 10, 64, 2, 4, 1, 0, 0, FAKE, None, None, None, None, None) == 2   # too many vectors
    assert Mp(FAKE, ctypes.c_void_p(0x1004), FAKE, 2, 4, 4, 64, 2, 4, 1, 0, 0, FAKE, None, None, None, None, None) == 3   # misaligned second gradient
    assert Mp(None, None, None, 0, 4, 4, 64, 2, 4, 1, 0, 0, None, None, None, None, None, None) == 0


def test_dgrad_rejects_bad_arguments_before_launch(lib):
    L, C = lib.sdgp_dgrad_linear, lib.sdgp_dgrad_conv2d
    ws = ctypes.c_void_p(0x10000)
    assert L(FAKE, FAKE, FAKE, 128, 256, 128, 2, 4, 1, 0, None, 0, 0, None) == 4        # no workspace
    need = lib.sdgp_workspace_size_linear(128, 256, 128, 0)
    assert need == 128 * 256 + 128 * 256 // 8
    assert L(FAKE, FAKE, FAKE, 128, 256, 128, 2, 4, 1, 0, ws, need - 1, 0, None) == 4   # short workspace
    assert L(FAKE, FAKE, FAKE, 128, 256, 128, 3, 4, 1, 0, ws, need, 0, None) == 2       # 3:4 not 2:4-compatible
    assert L(FAKE, FAKE, FAKE, 128, 256, 128, 2, 4, 1, 0, ws, need, 9, None) == 1       # unknown flags
    assert L(FAKE, FAKE, FAKE, 128, 250, 128, 2, 4, 1, 0, ws, need, 0, None) == 1       # K % m != 0
    assert L(None, FAKE, FAKE, 128, 256, 128, 2, 4, 1, 0, ws, need, 0, None) == 1
    assert L(FAKE, FAKE, FAKE, 0, 256, 128, 2, 4, 1, 0, None, 0, 0, None) == 0          # rows == 0: no-op
    assert C(FAKE, FAKE, FAKE, 2, 8, 8, 64, 128, 3, 3, 3, 1, 2, 4, 1, 0, ws, 1 << 30, 0, None) == 2  # stride 3
    assert C(FAKE, FAKE, FAKE, 2, 8, 8, 64, 128, 3, 3, 1, 1, 2, 4, 1, 0, None, 0, 0, None) == 4
    assert lib.sdgp_workspace_size_conv2d(2, 8, 8, 64, 128, 3, 3, 1, 1, 0) == 2 * 8 * 8 * 128 * 9 // 8
    assert lib.sdgp_workspace_size_conv2d(2, 8, 8, 64, 128, 3, 3, 1, 1, 2) == 0
    # masked mode: any n <= m, workspace = a dense copy of dL/dO
    assert lib.sdgp_workspace_size_linear(128, 256, 128, 3) == 128 * 256 * 2
    assert lib.sdgp_workspace_size_conv2d(2, 8, 8, 64, 128, 3, 3, 1, 1, 3) == 2 * 8 * 8 * 128 * 2
    assert L(FAKE, FAKE, FAKE, 128, 256, 128, 3, 4, 1, 0, None, 0, 3, None) == 4        # 3:4 masked: needs the workspace
    assert L(FAKE, FAKE, FAKE, 128, 256, 128, 3, 4, 1, 0, ws, 128 * 256 * 2 - 1, 3, None) == 4
    assert L(FAKE, FAKE, FAKE, 128, 256, 128, 5, 4, 1, 0, ws, 1 << 20, 3, None) == 1    # n > m
    assert L(FAKE, FAKE, FAKE, 128, 256, 128, 2, 4, 1, 0, ws, need, 5, None) == 1       # flags past the last mode
    # per-channel reading: compressed tensor + 3*K floats + a copy of W; scheme must be the rescaled one
    need_ch = need + 256 * 3 * 4 + 256 * 128 * 2
    assert lib.sdgp_workspace_size_linear(128, 256, 128, 4) == need_ch
    assert L(FAKE, FAKE, FAKE, 128, 256, 128, 2, 4, 2, 0, ws, need_ch - 1, 4, None) == 4
    assert L(FAKE, FAKE, FAKE, 128, 256, 128, 2, 4, 1, 0, ws, need_ch, 4, None) == 1     # magnitude scheme with the channel mode
    S = lib.sdgp_channel_scales
    assert S(FAKE, 4, 64, 2, 4, 7, FAKE, None) == 1      # unknown element type
    assert S(FAKE, 4, 66, 2, 4, 0, FAKE, None) == 1      # K % m != 0
    assert S(FAKE, 4, 64, 2, 4, 0, None, None) == 1      # no output


def test_static_scratch_variant_rejects_bad_arguments_before_launch(lib):
    """sdgp_dgrad_linear_static validates on the host: nothing below reaches a launch or the scratch lookup."""
    T = lib.sdgp_dgrad_linear_static
    T.restype = ctypes.c_int
    T.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int64] * 3 + [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_uint64,
                                                                ctypes.c_void_p]
    assert T(FAKE, FAKE, FAKE, 64, 192, 64, 2, 4, 1, 0, None) == 2                      # K % 128 != 0
    assert T(FAKE, FAKE, FAKE, 64, 256, 96, 2, 4, 1, 0, None) == 2                      # N % 64 != 0
    assert T(FAKE, FAKE, FAKE, 64, 256, 64, 3, 4, 1, 0, None) == 2                      # 3:4 has no compressed form
    assert T(FAKE, FAKE, FAKE, 64, 256, 64, 0, 4, 1, 0, None) == 1                      # n < 1
    assert T(FAKE, FAKE, FAKE, 64, 256, 64, 2, 4, 9, 0, None) == 1                      # unknown scheme
    assert T(ctypes.c_void_p(0x1008), FAKE, FAKE, 64, 256, 64, 2, 4, 1, 0, None) == 3   # misaligned dO
    assert T(FAKE, FAKE, ctypes.c_void_p(0x1004), 64, 256, 64, 2, 4, 1, 0, None) == 3   # misaligned dD
    assert T(None, FAKE, FAKE, 64, 256, 64, 2, 4, 1, 0, None) == 1                      # null input
    assert T(FAKE, FAKE, FAKE, 8193, 1024, 64, 2, 4, 1, 0, None) == 7                   # beyond the fixed scratch
    assert T(FAKE, FAKE, FAKE, 0, 256, 64, 2, 4, 1, 0, None) == 0                       # rows == 0: no-op
