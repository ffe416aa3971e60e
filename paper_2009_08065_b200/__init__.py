"""Block-structured pruning for BERT-family linear layers on NVIDIA B200 (sm_100a).

Thin Python binding over the C-ABI CUDA library `libbsp.so` (declared in include/bsp.h).
Every computation runs in the library's kernels; this package only marshals arguments.
torch is used for device memory and streams.
"""
from .binding import (  # noqa: F401
    BspError,
    ORIENT_C, ORIENT_R, PEN_L2, PEN_L2SQ, ACT_NONE, ACT_GELU,
    PackedMatrix, LayerJob, make_job_array, ChainOp, make_chain_array,
    lib, library_path,
    bsp_group_norms, bsp_penalty_grad, bsp_pack_bound, bsp_pack_scratch_bytes, bsp_prune_pack, bsp_prune_pack_static, bsp_percentile_threshold, bsp_apply_mask, bsp_prepare_batched, bsp_percentile_threshold_batched,
    bsp_linear_plan_bytes, bsp_linear_plan, bsp_linear_plan_t, bsp_linear_backward_weight, bsp_linear_planned, bsp_linear_planned_ex,
    LINEAR_AUTO, LINEAR_ONE_CTA, LINEAR_CTA_PAIR, LINEAR_PLAN_STABLE, LINEAR_OUT_TRANSPOSED, bsp_linear_gathered_ex, bsp_linear, bsp_linear_status, bsp_linear_chain, bsp_linear_chain_ws_bytes,
    bsp_linear_gather_plan_bytes, bsp_linear_gather_plan, bsp_transpose, bsp_linear_gathered,
    bsp_masked_adam_step, bsp_repack_values, bsp_dense_mask,
    bsp_linear_cuda_core, bsp_status_string, bsp_set_wait_limit_ms, bsp_wait_selftest,
    ROUTE_AUTO, ROUTE_ZERO_EXPANDED, ROUTE_GATHERED, make_linear_call, bsp_linear_route, bsp_linear_run, bsp_linear_tune,
)
