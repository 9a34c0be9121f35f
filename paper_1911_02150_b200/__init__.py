"""B200-native decode-attention step of multi-query attention (arXiv 1911.02150).

The product is the CUDA library ``libmqa_decode.so`` (C ABI: ``include/mqa_decode.h``);
this package is its thin Python binding plus the seeded synthetic workloads.
"""
from .binding import (  # noqa: F401
    MqaError, alloc_workspace, append_step_launches, kv_cache_append, lib, mha_decode_step, mha_decode_step_combine,
    mha_decode_step_split, mqa_decode_step, mqa_decode_step_combine, mqa_decode_step_noalloc, mqa_decode_append_step, mqa_decode_step_split, plan_splits, plan_kernel_name, set_wait_limit_cycles, set_test_withhold_copy, mqa_prefill_attention, prefill_workspace_bytes,
    status_string, workspace_bytes, mqa_layer_decode_step, layer_workspace_bytes, alloc_layer_workspace, mqa_decode_local_step, mqa_decode_append_step_host, host_staging_bytes, HostStep, AppendStep,
)
