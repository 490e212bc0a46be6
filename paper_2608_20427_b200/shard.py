"""Sequence-sharded BF1 prefill: one long sequence cut into contiguous shards of whole blocks, one
shard per rank (one process per GPU, `torch.distributed`).

The route is data independent (Section 3.1), so every rank can compute, without talking to anyone,
which of its key/value blocks each later rank reads (block 0, the blocks just in front of that rank's
shard, the dyadic predecessors of its query blocks: Proposition 1) and which blocks it will receive
itself.  The exchange is a set of plain point-to-point copies (NCCL send/recv on GPUs, gloo on CPUs)
that land in the receiver's own memory, in front of its own blocks; the attention kernel then runs on
that local tensor through a route that the library re-indexes on the device.  No collective, no
reduction: a shard's outputs depend on nothing else.

Only argument marshalling and communication calls live here; the plans and the attention are the
C-ABI library's (`bf1_shard_needed_blocks`, `bf1_plan_route_shard`, `bf1_attn_fwd`).
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch

from . import binding as B

BLOCK = 64


def shard_bounds(n_tokens: int, world: int) -> List[int]:
    """First block of every rank's shard (and one past the last): whole blocks, as even as they come."""
    nb = (n_tokens + BLOCK - 1) // BLOCK
    return [(nb * r) // world for r in range(world + 1)]


def exchange_plan(n_tokens: int, bounds: Sequence[int], cfg: Optional[B.RouteCfg] = None):
    """For every rank the ascending list of blocks it needs from earlier ranks (host only; every rank
    computes the same table).  Ranks with an empty shard need nothing."""
    return [B.shard_needed_blocks(n_tokens, bounds[r], bounds[r + 1], cfg) if bounds[r + 1] > bounds[r] else []
            for r in range(len(bounds) - 1)]


def owner_of(block: int, bounds: Sequence[int]) -> int:
    for r in range(len(bounds) - 1):
        if bounds[r] <= block < bounds[r + 1]:
            return r
    raise ValueError("block %d is outside the sequence" % block)


def exchange_kv(k_local: torch.Tensor, v_local: torch.Tensor, n_tokens: int, bounds: Sequence[int], rank: int,
                needed: Sequence[Sequence[int]], group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Send this rank's blocks to the later ranks that read them and receive the blocks this rank reads.

    k_local / v_local: this rank's own rows [own tokens, hkv, d] (its last block may be partial only on the last
    rank).  Returns the local "virtual sequence" tensors [len(needed[rank]) * 64 + own tokens, hkv, d]: the
    received blocks in ascending global order, then the own rows.  Received blocks land directly in their place.
    """
    import torch.distributed as dist
    world = len(bounds) - 1
    mine = list(needed[rank])
    own_tokens = k_local.shape[0]
    out = []
    for t in (k_local, v_local):
        virt = torch.empty((len(mine) * BLOCK + own_tokens,) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        virt[len(mine) * BLOCK:] = t
        out.append(virt)
    ops, keep = [], []
    # receives: one message per (source rank, tensor), covering that source's blocks, which are contiguous in the
    # ascending list because shards are contiguous
    pos = 0
    while pos < len(mine):
        src = owner_of(mine[pos], bounds)
        end = pos
        while end < len(mine) and owner_of(mine[end], bounds) == src:
            end += 1
        for virt in out:
            ops.append(dist.P2POp(dist.irecv, virt[pos * BLOCK:end * BLOCK], src, group))
        pos = end
    # sends: for every later rank, the blocks of mine it reads, gathered into one message per tensor
    lo = bounds[rank]
    for dst in range(rank + 1, world):
        blocks = [p for p in needed[dst] if bounds[rank] <= p < bounds[rank + 1]]
        if not blocks:
            continue
        rows = torch.cat([torch.arange((p - lo) * BLOCK, (p - lo + 1) * BLOCK) for p in blocks]).to(k_local.device)
        for t in (k_local, v_local):
            buf = t.index_select(0, rows).contiguous()
            keep.append(buf)
            ops.append(dist.P2POp(dist.isend, buf, dst, group))
    if ops:
        for req in dist.batch_isend_irecv(ops):
            req.wait()
    return out[0], out[1]


def shard_attn_fwd(q_local, k_local, v_local, n_tokens: int, rank: int, world: int, cfg: Optional[B.RouteCfg] = None,
                   scale: Optional[float] = None, group=None):
    """One rank's part of a sequence-sharded BF1 forward on CUDA tensors: plan, exchange, attention.
    Returns (o_local [own tokens, hq, d] bf16, lse_local [hq, own tokens] fp32, selected pairs of this shard)."""
    bounds = shard_bounds(n_tokens, world)
    needed = exchange_plan(n_tokens, bounds, cfg)
    lo, hi = bounds[rank], bounds[rank + 1]
    if hi <= lo:
        return q_local[:0], torch.empty((q_local.shape[1], 0), dtype=torch.float32, device=q_local.device), 0
    k_virt, v_virt = exchange_kv(k_local, v_local, n_tokens, bounds, rank, needed, group)
    front = len(needed[rank]) * BLOCK
    q_virt = torch.zeros((front + q_local.shape[0],) + tuple(q_local.shape[1:]), dtype=q_local.dtype, device=q_local.device)
    q_virt[front:] = q_local
    nb = torch.tensor(needed[rank], dtype=torch.int32, device=q_local.device)
    route, cu = B.plan_route_shard(n_tokens, lo, hi, nb, cfg)
    o, lse = B.attn_fwd(q_virt, k_virt, v_virt, cu, q_virt.shape[0], route, scale=scale)
    return o[front:], lse[:, front:], route
