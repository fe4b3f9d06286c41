"""Operator-split linear layer for NVIDIA B200: thin Python binding over the C-ABI library.

Every step of the path runs in the CUDA kernels of ``libosdp.so``; this package only
marshals arguments.  There is no CPU fallback: if the library is missing, loading it raises.
``paper_2209_13258_b200.inputs`` (seeded synthetic inputs) does not need the library.
"""
from .binding import (  # noqa: F401
    ACT_GELU_ERF, ACT_GELU_TANH, ACT_NONE, DTYPE_BF16, DTYPE_FP32, FLAG_ACCUMULATE_DW, FLAG_CARRY_BF16, FLAG_RECOMPUTE, FLAG_PAIR_SLICES, FLAG_SLICE_MAJOR, OP_LINEAR_BWD, OP_LINEAR_FWD,
    OP_MLP_BWD, OP_MLP_FWD, SPLIT_OUT, SPLIT_RED, OsdpError, lib, lib_path,
    osdp_last_cuda_error, osdp_read_device_status, osdp_slice_range, osdp_split_linear_bwd,
    osdp_split_linear_bwd_slice, osdp_split_linear_fwd, osdp_split_linear_fwd_slice,
    osdp_split_linear_workspace_bytes, osdp_split_mlp_bwd, osdp_split_mlp_fwd, osdp_status_string,
    osdp_version, new_workspace, osdp_bias_grad_noalloc, osdp_debug_wait_probe, osdp_suggest_granularity,
    osdp_zdp_shard_layout, osdp_zdp_linear_fwd_slice, osdp_zdp_linear_bwd_slice,
    osdp_plan_cost, osdp_plan_search, osdp_plan_expand_slices, osdp_plan_search_granularity,
    osdp_split_linear_fwd_f8, osdp_split_linear_bwd_f8, osdp_zdp_linear_bwd_slice_scatter,
    osdp_zdp_mlp_fwd_slice, osdp_zdp_mlp_bwd_slice,
)
