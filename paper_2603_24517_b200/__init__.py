"""B200 (sm_100a) fused attention forward: BF16, head dim 128, MHA and GQA, causal or not,
with per-row log-sum-exp.  The computation lives in ``libattn_b200.so`` (hand-written CUDA,
C ABI in ``include/attn.h``); this package is its ctypes binding."""
from .binding import (AttnError, attention_forward, attn_fwd, attn_fwd_host, attn_fwd_noalloc, attn_fwd_noalloc_status, attn_fwd_status, attn_fwd_strided, attn_fwd_strided_status,  # noqa: F401
                      attn_fwd_splitkv, attn_fwd_splitkv_status, attn_last_device_status, attn_last_launch_clock, attn_launch_clocks, attn_merge, attn_merge_n, attn_merge_status,
                      attn_splitkv_workspace_bytes, attn_plan, attn_plan_item, attn_plan_item_pair, attn_release_host_staging, attn_selftest_wait_timeout, attn_set_option, attn_get_option, OPTION_DEFAULTS,
                      attn_status_str, attn_version, load_library)
