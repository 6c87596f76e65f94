"""SDGP hot path for NVIDIA B200 (sm_100a): N:M pruning of the output data gradient and the
sparse tensor-core data-gradient contraction, behind the C ABI declared in ``include/sdgp.h``."""
from .binding import (BF16, FP16, FLAG_CHANNEL, FLAG_DENSE, FLAG_FUSED, FLAG_MASKED, FLAG_TWO_PASS, MAGNITUDE, RANDOM, RESCALED_MAGNITUDE,  # noqa: F401
                      SdgpError, sdgp_dgrad_conv2d, sdgp_dgrad_linear, sdgp_dgrad_linear_static, sdgp_last_device_error, sdgp_prune, sdgp_selftest_bounded_wait,
                      sdgp_spmm_conv2d, sdgp_spmm_linear, sdgp_prune_typed, sdgp_dgrad_linear_typed, sdgp_dgrad_conv2d_typed,
                      sdgp_spmm_linear_typed, sdgp_spmm_conv2d_typed, sdgp_channel_scales, sdgp_relu_backward_prune, sdgp_residual_relu_backward_prune, sdgp_maxpool_relu_backward_prune, sdgp_workspace_size_conv2d,
                      sdgp_workspace_size_conv2d_grouped, sdgp_dgrad_conv2d_grouped,
                      sdgp_workspace_size_linear, status_string)
