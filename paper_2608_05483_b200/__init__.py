"""B200 (sm_100a) batched heterogeneous-adapter LoRA delta: Python binding of the C ABI.

The product is the CUDA shared library built from csrc/ (declared in include/plora.h);
this package only loads it and marshals arguments.
"""
from .binding import (  # noqa: F401
    EXPORTS, OK, ERR_BAD_ADAPTER_ID, ERR_DEBUG_CHECK, ERR_CUDA, ERR_INVALID_ARG, ERR_NOT_REGISTERED, ERR_TIMEOUT, ERR_UNSUPPORTED,
    ERR_WORKSPACE, PATH_AUTO, PATH_FUSED, PATH_SGMV, PATH_SGMV_SPLIT, PATH_UNFUSED, Context, PloraError, PoolDesc, library_path, load,
    plora_bucket, plora_bucket_view, plora_cost_model, plora_create, plora_destroy, plora_device_status, plora_expand, plora_expand_m16,
    plora_launch_count, plora_lora_delta, plora_lora_delta_group, plora_lora_delta_host, plora_lora_delta_host_async, plora_host_sync, plora_lora_delta_noalloc, plora_pool_max_rank, plora_pool_slab_bytes,
    plora_register_pool, plora_set_path, plora_shrink, plora_shrink_m16, status_string,
    attn_decode, plora_attn_decode, plora_attn_set_debug, plora_attn_status, plora_attn_workspace_bytes,
    plora_set_test_hook, plora_set_wait_limit, plora_set_inputs_resident, plora_stream_read, HOOK_NONE, HOOK_WITHHOLD_RELEASE, HOOK_MAX_CYCLES,
)
