"""B200-native low-rank pre-factorized layers (Pufferfish hot path).

The product is ``libpf.so`` (CUDA kernels for sm_100a behind the C ABI of ``include/pf.h``);
this package is the thin Python binding over it.  There is no CPU fallback: importing the
binding without the built library raises.
"""
from .binding import (  # noqa: F401
    PF_ACT_NONE, PF_ACT_RELU, PF_BF16, PF_F32, PF_GRAD_ACCUMULATE, PF_GRAD_F32, PfError, lib, pf_bias_act_bwd, pf_last_device_status, pf_launch_count, pf_lowrank_conv_bwd,
    pf_lowrank_conv_fwd, pf_lowrank_conv_workspace, pf_lowrank_linear_bwd,
    pf_lowrank_linear_fwd, pf_lowrank_linear_fwd_act, pf_lowrank_linear_fwd_static, pf_lowrank_linear_grouped_bwd,
    pf_lowrank_linear_grouped_fwd, pf_lowrank_linear_grouped_workspace, pf_lowrank_linear_workspace, pf_pack_factor_grads,
    pf_static_scratch_bytes, pf_status_string, pf_unpack_factor_grads, pf_version)
