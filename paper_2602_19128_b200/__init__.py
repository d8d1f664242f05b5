"""B200-native fused Mixture-of-Experts layer forward (router, sort-scatter, grouped gate/up GEMM
with SwiGLU, grouped down GEMM, weighted combine) behind a C-ABI library; see ``include/moe.h``."""
from .binding import (MOE_FLAG_NONE, MOE_FLAG_VALIDATION_GEMM, MOE_FLAG_SINGLE_CTA_GEMM, MOE_FLAG_TWO_SLAB_GEMM, MOE_FLAG_NARROW_TILES, MOE_FLAG_GATHER_IN_LOAD, MOE_OK, MoeError, alloc_workspace, lib,  # noqa: F401
                      moe_forward, moe_forward_local, moe_route_grouped, moe_forward_grouped, grouped_router, GroupedRouter, moe_forward_fp8w, moe_forward_mxfp8, moe_forward_mxfp8_host, moe_mxfp8_pack_scales, moe_mxfp8_quantize_rows, moe_mxfp8_workspace_bytes, moe_mxfp8_workspace_layout, mx_workspace_views, moe_forward_host, moe_forward_staged, make_stage_events, STAGE_NAMES, moe_forward_launch_count, moe_token_tile_rows, moe_last_status, moe_selftest_wait_timeout, moe_route, moe_route_static,
                      moe_route_workspace_bytes, moe_status_string, moe_workspace_bytes, moe_workspace_layout,
                      workspace_views, gqa_decode_workspace_bytes, gqa_decode_split_tokens, gqa_paged_decode,
                      gqa_selftest_wait_timeout)
