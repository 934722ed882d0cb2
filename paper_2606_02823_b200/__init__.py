"""B200-native (sm_100a) library for the rotated W2A4 / W4A4 quantized linear layer of Qift.

The product is the C-ABI shared library built from csrc/ (declared in include/qift.h); this package
is its thin Python binding.  Importing the package does not load the library; the first call does,
and raises if it has not been built.
"""
from .binding import *  # noqa: F401,F403
from .binding import (lib, status_string, QiftError, qift_packed_bytes, qift_workspace_bytes, qift_pack_weights,
                      qift_unpack_codes, qift_rotate, qift_quantize_act, qift_w2a4_linear, qift_w4a4_linear, qift_w3a4_linear,
                      qift_linear_route, qift_device_status, qift_forward_scratch_bytes, qift_forward,
                      qift_forward_host, qift_group_plan_bytes, qift_group_plan, qift_group_quantize_act,
                      qift_group_linear, qift_group_forward, qift_group_forward_host, GroupPlan, qift_static_scratch_bytes,
                      qift_w2a4_linear_static, Kv4Cache, KV_KEYS, KV_VALUES, qift_kv4_quantize, qift_kv4_attention_workspace_bytes,
                      qift_kv4_attention_decode, qift_expand_weights, qift_expanded_linear, qift_diag_grid_quantize,
                      qift_diag_bucket_stats, qift_diag_ratio_scan_workspace_bytes, qift_diag_ratio_scan,
                      qift_selftest_wait_timeout, qift_levels_bytes, qift_forward_multi, qift_linear_multi)
