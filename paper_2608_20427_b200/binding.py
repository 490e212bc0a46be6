"""Thin Python binding of the BF1 C-ABI library (argument marshalling only).

Every step of the operator runs in the library's CUDA kernels.  PyTorch is used for device
memory, streams and nothing else.  There is no CPU or PyTorch fallback: if the shared
library cannot be built or loaded, importing callers get an exception.
"""
from __future__ import annotations

import ctypes
import math
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

from . import build as _build

BF1_OK = 0
DEV_BAD_SEQLENS, DEV_CAPACITY, DEV_WAIT_TIMEOUT, DEV_BAD_ROUTE = 1, 2, 4, 8

EXPORTS = ("bf1_route_capacity", "bf1_plan_route", "bf1_attn_fwd", "bf1_dense_causal_fwd",
           "bf1_attn_fwd_noalloc", "bf1_plan_decode", "bf1_decode_workspace_bytes", "bf1_decode_fwd",
           "bf1_attn_bwd", "bf1_attn_bwd_workspace_bytes", "bf1_shard_needed_blocks", "bf1_plan_route_shard",
           "bf1_shard_needed_blocks_strided", "bf1_plan_route_shard_strided",
           "bf1_last_error", "bf1_version")


class RouteCfg(ctypes.Structure):
    """Mirror of bf1_route_cfg.  Defaults: the paper's reported configuration (Section 3.1)."""
    _fields_ = [("block", ctypes.c_int32), ("local_blocks", ctypes.c_int32),
                ("global_first", ctypes.c_int32), ("dyadic", ctypes.c_int32)]

    def __init__(self, block: int = 64, local_blocks: int = 2, global_first: int = 1, dyadic: int = 1):
        super().__init__(block, local_blocks, global_first, dyadic)


class _RouteC(ctypes.Structure):
    """Mirror of bf1_route."""
    _fields_ = [("capacity_qblocks", ctypes.c_int32), ("max_degree", ctypes.c_int32),
                ("qb_seq", ctypes.c_void_p), ("qb_block", ctypes.c_void_p),
                ("kv_count", ctypes.c_void_p), ("kv_idx", ctypes.c_void_p),
                ("pair_count", ctypes.c_void_p), ("order", ctypes.c_void_p),
                ("total_pairs", ctypes.c_void_p), ("num_qblocks", ctypes.c_void_p),
                ("status", ctypes.c_void_p), ("sched", ctypes.c_void_p)]


class _DecodePlanC(ctypes.Structure):
    """Mirror of bf1_decode_plan."""
    _fields_ = [("max_degree", ctypes.c_int32), ("count", ctypes.c_void_p), ("page", ctypes.c_void_p),
                ("block", ctypes.c_void_p), ("status", ctypes.c_void_p)]


class Bf1Error(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("bf1 error %d: %s" % (code, msg))
        self.code = code


_lib = None


def load():
    """Load (building first if needed) libbf1.so and declare its signatures."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    L = ctypes.CDLL(path)
    i32, i64, vp, f32 = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p, ctypes.c_float
    L.bf1_route_capacity.restype = ctypes.c_int
    L.bf1_route_capacity.argtypes = [i32, i64, i32, ctypes.POINTER(RouteCfg), ctypes.POINTER(i32), ctypes.POINTER(i32)]
    L.bf1_plan_route.restype = ctypes.c_int
    L.bf1_plan_route.argtypes = [vp, i32, i64, i32, ctypes.POINTER(RouteCfg), ctypes.POINTER(_RouteC), vp]
    L.bf1_attn_fwd.restype = ctypes.c_int
    L.bf1_attn_fwd.argtypes = [vp, vp, vp, vp, i32, i64, i32, i32, i32, i32, f32, ctypes.POINTER(_RouteC), vp, vp, vp]
    L.bf1_dense_causal_fwd.restype = ctypes.c_int
    L.bf1_dense_causal_fwd.argtypes = [vp, vp, vp, vp, i32, i64, i32, i32, i32, i32, f32, vp, vp, vp, vp]
    L.bf1_attn_fwd_noalloc.restype = ctypes.c_int
    L.bf1_attn_fwd_noalloc.argtypes = [vp, vp, vp, vp, i32, i64, i32, i32, i32, i32, f32, ctypes.POINTER(RouteCfg),
                                       vp, vp, vp, vp]
    L.bf1_plan_decode.restype = ctypes.c_int
    L.bf1_plan_decode.argtypes = [vp, vp, i32, i32, ctypes.POINTER(RouteCfg), ctypes.POINTER(_DecodePlanC), vp]
    L.bf1_decode_workspace_bytes.restype = i64
    L.bf1_decode_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
    L.bf1_decode_fwd.restype = ctypes.c_int
    L.bf1_decode_fwd.argtypes = [vp, vp, vp, i32, vp, i32, i32, i32, i32, f32, ctypes.POINTER(_DecodePlanC), vp, vp,
                                 vp, vp]
    L.bf1_attn_bwd_workspace_bytes.restype = i64
    L.bf1_attn_bwd_workspace_bytes.argtypes = [ctypes.POINTER(_RouteC), i64, i32, i32, i32]
    L.bf1_attn_bwd.restype = ctypes.c_int
    L.bf1_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i64, i32, i32, i32, i32, f32, ctypes.POINTER(_RouteC),
                               vp, vp, vp, vp, vp]
    L.bf1_shard_needed_blocks.restype = ctypes.c_int
    L.bf1_shard_needed_blocks.argtypes = [i64, ctypes.POINTER(RouteCfg), i32, i32, ctypes.POINTER(i32), i32, ctypes.POINTER(i32)]
    L.bf1_plan_route_shard.restype = ctypes.c_int
    L.bf1_plan_route_shard.argtypes = [i64, i32, i32, ctypes.POINTER(RouteCfg), vp, i32, ctypes.POINTER(_RouteC), vp, vp]
    L.bf1_shard_needed_blocks_strided.restype = ctypes.c_int
    L.bf1_shard_needed_blocks_strided.argtypes = [i64, ctypes.POINTER(RouteCfg), i32, i32, i32, ctypes.POINTER(i32), i32,
                                                  ctypes.POINTER(i32)]
    L.bf1_plan_route_shard_strided.restype = ctypes.c_int
    L.bf1_plan_route_shard_strided.argtypes = [i64, i32, i32, i32, ctypes.POINTER(RouteCfg), vp, i32, ctypes.POINTER(_RouteC),
                                               vp, vp]
    L.bf1_last_error.restype = ctypes.c_char_p
    L.bf1_last_error.argtypes = []
    L.bf1_version.restype = ctypes.c_int
    _lib = L
    return L


def _check(rc: int):
    if rc != BF1_OK:
        raise Bf1Error(rc, load().bf1_last_error().decode())


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def route_capacity(batch: int, total_tokens: int, max_seqlen: int, cfg: Optional[RouteCfg] = None):
    """(capacity_qblocks, max_degree) for a batch; host only."""
    cfg = cfg or RouteCfg()
    cap, deg = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(load().bf1_route_capacity(batch, total_tokens, max_seqlen, ctypes.byref(cfg),
                                     ctypes.byref(cap), ctypes.byref(deg)))
    return cap.value, deg.value


@dataclass
class Route:
    """Device arrays of a planned route plus the C struct that points at them."""
    cfg: RouteCfg
    capacity_qblocks: int
    max_degree: int
    qb_seq: torch.Tensor
    qb_block: torch.Tensor
    kv_count: torch.Tensor
    kv_idx: torch.Tensor
    pair_count: torch.Tensor
    order: torch.Tensor
    total_pairs: torch.Tensor
    num_qblocks: torch.Tensor
    status: torch.Tensor
    sched: torch.Tensor
    c: _RouteC = None

    @staticmethod
    def empty(capacity_qblocks: int, max_degree: int, device, cfg: Optional[RouteCfg] = None) -> "Route":
        i32 = dict(dtype=torch.int32, device=device)
        r = Route(cfg=cfg or RouteCfg(), capacity_qblocks=capacity_qblocks, max_degree=max_degree,
                  qb_seq=torch.empty(capacity_qblocks, **i32), qb_block=torch.empty(capacity_qblocks, **i32),
                  kv_count=torch.empty(capacity_qblocks, **i32),
                  kv_idx=torch.empty((capacity_qblocks, max_degree), **i32),
                  pair_count=torch.empty(capacity_qblocks, **i32), order=torch.empty(capacity_qblocks, **i32),
                  total_pairs=torch.zeros(1, dtype=torch.int64, device=device),
                  num_qblocks=torch.zeros(1, **i32), status=torch.zeros(1, **i32),
                  sched=torch.zeros(2, **i32))
        r.c = _RouteC(capacity_qblocks, max_degree, r.qb_seq.data_ptr(), r.qb_block.data_ptr(),
                      r.kv_count.data_ptr(), r.kv_idx.data_ptr(), r.pair_count.data_ptr(), r.order.data_ptr(),
                      r.total_pairs.data_ptr(), r.num_qblocks.data_ptr(), r.status.data_ptr(),
                      r.sched.data_ptr())
        return r

    @staticmethod
    def from_host(qb_seq, qb_block, kv_count, kv_idx, pair_count, order, total_pairs: int, device,
                  cfg: Optional[RouteCfg] = None) -> "Route":
        """Upload a route the caller built on the host (any ascending lists whose last entry is the
        query block itself; kv_idx [slots, max_degree] padded with -1).  Marshalling only."""
        kv_idx = torch.as_tensor(kv_idx, dtype=torch.int32)
        slots, max_degree = kv_idx.shape
        r = Route.empty(max(slots, 1), max_degree, device, cfg)
        for name, src in (("qb_seq", qb_seq), ("qb_block", qb_block), ("kv_count", kv_count),
                          ("pair_count", pair_count), ("order", order)):
            getattr(r, name)[:slots].copy_(torch.as_tensor(src, dtype=torch.int32))
        r.kv_idx[:slots].copy_(kv_idx)
        r.total_pairs.fill_(int(total_pairs))
        r.num_qblocks.fill_(slots)
        return r

    def check_status(self):
        """Synchronising read of the device status word; raises if any BF1_DEV_* bit is set."""
        st = int(self.status.item())
        if st:
            raise Bf1Error(-100, "device status 0x%x" % st)


def plan_route(cu_seqlens: torch.Tensor, max_seqlen: int, cfg: Optional[RouteCfg] = None,
               route: Optional[Route] = None, stream=None) -> Route:
    """bf1_plan_route: Eq. 1 lists for every query block of the packed batch."""
    cfg = cfg or RouteCfg()
    assert cu_seqlens.is_cuda and cu_seqlens.dtype == torch.int32 and cu_seqlens.is_contiguous()
    batch = cu_seqlens.numel() - 1
    total = getattr(cu_seqlens, "_bf1_total", None)
    if total is None:
        total = int(cu_seqlens[-1].item())
    if route is None:
        cap, deg = route_capacity(batch, total, max_seqlen, cfg)
        route = Route.empty(cap, deg, cu_seqlens.device, cfg)
    _check(load().bf1_plan_route(cu_seqlens.data_ptr(), batch, total, max_seqlen, ctypes.byref(cfg),
                                 ctypes.byref(route.c), _stream_ptr(stream)))
    route.cfg = cfg
    return route


def _check_qkv(q, k, v):
    for t in (q, k, v):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and t.dim() == 3
    T, hq, d = q.shape
    assert k.shape == v.shape and k.shape[0] == T and k.shape[2] == d
    return T, hq, k.shape[1], d


def attn_fwd(q, k, v, cu_seqlens, max_seqlen: int, route: Route, scale: Optional[float] = None,
             out=None, lse=None, stream=None):
    """bf1_attn_fwd.  q [T, hq, d], k/v [T, hkv, d] bf16 CUDA -> (o [T, hq, d] bf16, lse [hq, T] fp32)."""
    T, hq, hkv, d = _check_qkv(q, k, v)
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((hq, T), dtype=torch.float32, device=q.device)
    _check(load().bf1_attn_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), cu_seqlens.data_ptr(),
                               cu_seqlens.numel() - 1, T, max_seqlen, hq, hkv, d,
                               float(scale) if scale else 0.0, ctypes.byref(route.c), out.data_ptr(),
                               lse.data_ptr(), _stream_ptr(stream)))
    return out, lse


def dense_causal_fwd(q, k, v, cu_seqlens, max_seqlen: int, scale: Optional[float] = None, out=None,
                     lse=None, work=None, stream=None):
    """bf1_dense_causal_fwd: plain causal attention through the same kernel.  `work`: optional
    zero-initialised int32[4] CUDA tensor (word 0 = device status, words 1..2 = hand-out counters)."""
    T, hq, hkv, d = _check_qkv(q, k, v)
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((hq, T), dtype=torch.float32, device=q.device)
    _check(load().bf1_dense_causal_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), cu_seqlens.data_ptr(),
                                       cu_seqlens.numel() - 1, T, max_seqlen, hq, hkv, d,
                                       float(scale) if scale else 0.0, out.data_ptr(), lse.data_ptr(),
                                       work.data_ptr() if work is not None else None,
                                       _stream_ptr(stream)))
    return out, lse


def attn_fwd_noalloc(q, k, v, cu_seqlens, max_seqlen: int, out, lse, cfg: Optional[RouteCfg] = None,
                     scale: Optional[float] = None, status=None, stream=None):
    """bf1_attn_fwd_noalloc: plan + attention using the library's built-in scratch array.

    For callers that must not allocate device memory, so `out` and `lse` are required here and
    the call itself allocates nothing (neither through torch nor through CUDA).  Up to 4096
    query blocks per batch; calls sharing a GPU must not overlap in time."""
    T, hq, hkv, d = _check_qkv(q, k, v)
    cfg = cfg or RouteCfg()
    total = getattr(cu_seqlens, "_bf1_total", T)
    _check(load().bf1_attn_fwd_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), cu_seqlens.data_ptr(),
                                       cu_seqlens.numel() - 1, total, max_seqlen, hq, hkv, d,
                                       float(scale) if scale else 0.0, ctypes.byref(cfg), out.data_ptr(),
                                       lse.data_ptr(), status.data_ptr() if status is not None else None,
                                       _stream_ptr(stream)))
    return out, lse


@dataclass
class DecodePlan:
    """Device arrays of a decode plan (one page list per sequence) plus the C struct."""
    max_degree: int
    count: torch.Tensor
    page: torch.Tensor
    block: torch.Tensor
    status: torch.Tensor
    c: _DecodePlanC = None

    @staticmethod
    def empty(batch: int, max_degree: int, device) -> "DecodePlan":
        i32 = dict(dtype=torch.int32, device=device)
        p = DecodePlan(max_degree, torch.zeros(batch, **i32), torch.full((batch, max_degree), -1, **i32),
                       torch.zeros(batch, **i32), torch.zeros(1, **i32))
        p.c = _DecodePlanC(max_degree, p.count.data_ptr(), p.page.data_ptr(), p.block.data_ptr(), p.status.data_ptr())
        return p


def plan_decode(seqlens: torch.Tensor, page_table: torch.Tensor, cfg: Optional[RouteCfg] = None,
                plan: Optional[DecodePlan] = None, stream=None) -> DecodePlan:
    """bf1_plan_decode: page list of the newest token's block for every sequence."""
    cfg = cfg or RouteCfg()
    assert seqlens.is_cuda and seqlens.dtype == torch.int32 and page_table.dtype == torch.int32
    batch, max_pages = page_table.shape
    if plan is None:
        _, deg = route_capacity(1, max_pages * 64, max_pages * 64, cfg)
        plan = DecodePlan.empty(batch, deg, seqlens.device)
    _check(load().bf1_plan_decode(seqlens.data_ptr(), page_table.data_ptr(), max_pages, batch, ctypes.byref(cfg),
                                  ctypes.byref(plan.c), _stream_ptr(stream)))
    return plan


def decode_workspace(batch: int, hq: int, hkv: int, max_degree: int, d: int, device) -> torch.Tensor:
    """Zero-initialised scratch for decode_fwd (reusable across calls that do not overlap)."""
    nbytes = int(load().bf1_decode_workspace_bytes(batch, hq, hkv, max_degree, d))
    return torch.zeros(max(nbytes, 16), dtype=torch.uint8, device=device)


def decode_fwd(q, k_pages, v_pages, seqlens, plan: DecodePlan, workspace, scale: Optional[float] = None,
               out=None, lse=None, stream=None):
    """bf1_decode_fwd.  q [batch, hq, d]; k_pages / v_pages [pages, 64, hkv, d] bf16 CUDA."""
    batch, hq, d = q.shape
    num_pages, page, hkv, d2 = k_pages.shape
    assert page == 64 and d2 == d and v_pages.shape == k_pages.shape
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((hq, batch), dtype=torch.float32, device=q.device)
    _check(load().bf1_decode_fwd(q.data_ptr(), k_pages.data_ptr(), v_pages.data_ptr(), num_pages, seqlens.data_ptr(),
                                 batch, hq, hkv, d, float(scale) if scale else 0.0, ctypes.byref(plan.c),
                                 workspace.data_ptr(), out.data_ptr(), lse.data_ptr(), _stream_ptr(stream)))
    return out, lse


def bwd_workspace(route: Route, total_tokens: int, hq: int, hkv: int, d: int, device) -> torch.Tensor:
    """Scratch for attn_bwd (reusable; its contents do not matter on entry)."""
    nbytes = int(load().bf1_attn_bwd_workspace_bytes(ctypes.byref(route.c), total_tokens, hq, hkv, d))
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def attn_bwd(q, k, v, o, lse, d_o, cu_seqlens, max_seqlen: int, route: Route, scale: Optional[float] = None,
             workspace=None, stream=None):
    """bf1_attn_bwd: (dq, dk, dv) in bf16 for the upstream gradient d_o; d = 128 only."""
    T, hq, hkv, d = _check_qkv(q, k, v)
    assert d_o.shape == q.shape and d_o.dtype == torch.bfloat16 and d_o.is_contiguous()
    if workspace is None:
        workspace = bwd_workspace(route, T, hq, hkv, d, q.device)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    _check(load().bf1_attn_bwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), d_o.data_ptr(),
                               cu_seqlens.data_ptr(), cu_seqlens.numel() - 1, T, max_seqlen, hq, hkv, d,
                               float(scale) if scale else 0.0, ctypes.byref(route.c), workspace.data_ptr(),
                               dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), _stream_ptr(stream)))
    return dq, dk, dv


def shard_needed_blocks(n_tokens: int, lo_block: int, hi_block: int, cfg: Optional[RouteCfg] = None):
    """bf1_shard_needed_blocks: ascending global KV blocks the shard [lo_block, hi_block) reads but does not own (host only)."""
    cfg = cfg or RouteCfg()
    cap = max(lo_block, 1)
    buf = (ctypes.c_int32 * cap)()
    count = ctypes.c_int32(0)
    _check(load().bf1_shard_needed_blocks(n_tokens, ctypes.byref(cfg), lo_block, hi_block, buf, cap, ctypes.byref(count)))
    return list(buf[:count.value])


def plan_route_shard(n_tokens: int, lo_block: int, hi_block: int, needed_blocks: torch.Tensor,
                     cfg: Optional[RouteCfg] = None, route: Optional[Route] = None, stream=None):
    """bf1_plan_route_shard: the shard's route over its local [needed | own] key/value tensor.
    Returns (route, cu_seqlens [2] int32 device tensor of the shard's virtual sequence)."""
    cfg = cfg or RouteCfg()
    assert needed_blocks.dtype == torch.int32 and needed_blocks.is_cuda
    if route is None:
        _, deg = route_capacity(1, n_tokens, n_tokens, cfg)
        route = Route.empty(hi_block - lo_block, deg, needed_blocks.device, cfg)
    cu = torch.zeros(2, dtype=torch.int32, device=needed_blocks.device)
    _check(load().bf1_plan_route_shard(n_tokens, lo_block, hi_block, ctypes.byref(cfg),
                                       needed_blocks.data_ptr() if needed_blocks.numel() else None, needed_blocks.numel(),
                                       ctypes.byref(route.c), cu.data_ptr(), _stream_ptr(stream)))
    own_tokens = min(n_tokens, hi_block * 64) - lo_block * 64
    cu._bf1_total = needed_blocks.numel() * 64 + own_tokens
    route.cfg = cfg
    return route, cu


def shard_needed_blocks_strided(n_tokens: int, first_block: int, stride: int, num_blocks: int,
                                cfg: Optional[RouteCfg] = None):
    """bf1_shard_needed_blocks_strided: ascending global KV blocks read but not owned by the shard
    first_block, first_block + stride, ... (num_blocks of them); host only."""
    cfg = cfg or RouteCfg()
    cap = max(first_block + (num_blocks - 1) * stride, 1)
    buf = (ctypes.c_int32 * cap)()
    count = ctypes.c_int32(0)
    _check(load().bf1_shard_needed_blocks_strided(n_tokens, ctypes.byref(cfg), first_block, stride, num_blocks, buf, cap,
                                                  ctypes.byref(count)))
    return list(buf[:count.value])


def plan_route_shard_strided(n_tokens: int, first_block: int, stride: int, num_blocks: int, needed_blocks: torch.Tensor,
                             cfg: Optional[RouteCfg] = None, route: Optional[Route] = None, stream=None):
    """bf1_plan_route_shard_strided: the strided shard's route over its local [needed | own] key/value tensor.
    Returns (route, cu_seqlens [2] int32 device tensor of the shard's virtual sequence)."""
    cfg = cfg or RouteCfg()
    assert needed_blocks.dtype == torch.int32 and needed_blocks.is_cuda
    if route is None:
        _, deg = route_capacity(1, n_tokens, n_tokens, cfg)
        route = Route.empty(num_blocks, deg, needed_blocks.device, cfg)
    cu = torch.zeros(2, dtype=torch.int32, device=needed_blocks.device)
    _check(load().bf1_plan_route_shard_strided(n_tokens, first_block, stride, num_blocks, ctypes.byref(cfg),
                                               needed_blocks.data_ptr() if needed_blocks.numel() else None,
                                               needed_blocks.numel(), ctypes.byref(route.c), cu.data_ptr(),
                                               _stream_ptr(stream)))
    last = first_block + (num_blocks - 1) * stride
    own_tokens = (num_blocks - 1) * 64 + min(64, n_tokens - last * 64)
    cu._bf1_total = needed_blocks.numel() * 64 + own_tokens
    route.cfg = cfg
    return route, cu


def cu_seqlens_tensor(seqlens: Sequence[int], device) -> torch.Tensor:
    cu = [0]
    for n in seqlens:
        cu.append(cu[-1] + int(n))
    t = torch.tensor(cu, dtype=torch.int32, device=device)
    t._bf1_total = cu[-1]   # host copy of the total, saves a device sync in plan_route
    return t


def default_scale(d: int) -> float:
    return 1.0 / math.sqrt(d)
