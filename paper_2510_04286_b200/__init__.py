"""B200-native (sm_100a) forward pass (and a first backward) of a SliceMoE layer behind a C ABI.

The compute lives in libslicemoe.so (CUDA kernels, built in-tree by
``python -m paper_2510_04286_b200.build``); this package only marshals arguments.
"""
from .binding import (  # noqa: F401
    ACT_GELU_TANH, ACT_RELU, BF16, F32, STAGES, Config, SliceMoEError, StageEvents, alloc_workspace,
    slicemoe_combine, slicemoe_dispatch, slicemoe_dispatch_static, slicemoe_expert_ffn, slicemoe_forward, slicemoe_forward_host, slicemoe_gate_dropout,
    slicemoe_forward_profiled, slicemoe_last_status, slicemoe_launch_count, slicemoe_load_stats, slicemoe_permute_columns, slicemoe_route,
    slicemoe_status_string, slicemoe_workspace_bytes, torch_dtype, slicemoe_backward, slicemoe_backward_workspace_bytes,
)
