"""BF1 causal dyadic block-sparse attention forward for B200 (sm_100a).

The product is the C-ABI library ``libbf1.so`` (sources under ``csrc/``, declarations in
``include/bf1.h``); this package is its Python binding.
"""
from .binding import (Bf1Error, attn_bwd, bwd_workspace, DecodePlan, decode_fwd, decode_workspace, plan_decode, Route, RouteCfg, attn_fwd, attn_fwd_noalloc, cu_seqlens_tensor, default_scale,
                      dense_causal_fwd, load, plan_route, plan_route_shard, plan_route_shard_strided, route_capacity, shard_needed_blocks,
                      shard_needed_blocks_strided)

__all__ = ["Bf1Error", "attn_bwd", "bwd_workspace", "DecodePlan", "decode_fwd", "decode_workspace", "plan_decode", "Route", "RouteCfg", "attn_fwd", "attn_fwd_noalloc", "cu_seqlens_tensor", "default_scale",
           "dense_causal_fwd", "load", "plan_route", "plan_route_shard", "plan_route_shard_strided", "route_capacity", "shard_needed_blocks",
           "shard_needed_blocks_strided"]
