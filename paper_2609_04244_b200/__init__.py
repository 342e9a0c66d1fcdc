"""B200-native fused routed-MoE decode step (one persistent sm_100a kernel) behind a C ABI.

`binding` mirrors the C entry points of include/moe_b200.h one to one; `workloads` holds the
seeded synthetic inputs.  There is no CPU fallback: without the compiled CUDA library and a
B200 every compute entry point raises.
"""
from .binding import (MoEError, MoEPlan, lib_path, load_library, moe_forward, moe_forward_debug, moe_forward_host, moe_forward_noalloc, moe_plan,  # noqa: F401
                      moe_plan_destroy, moe_plan_info, moe_tokens_per_launch, moe_plan_set_knob, moe_plan_get_knob, KNOBS, moe_sync_status, moe_workspace_bytes, moe_workspace_init,
                      SCORE_SIGMOID_BIAS, SCORE_SOFTMAX)

__all__ = ["MoEError", "MoEPlan", "lib_path", "load_library", "moe_forward", "moe_forward_debug", "moe_forward_host", "moe_forward_noalloc", "moe_plan",
           "moe_plan_destroy", "moe_plan_info", "moe_tokens_per_launch", "moe_plan_set_knob", "moe_plan_get_knob", "KNOBS", "moe_sync_status", "moe_workspace_bytes", "moe_workspace_init",
           "SCORE_SIGMOID_BIAS", "SCORE_SOFTMAX"]
