"""Sequence-sharded BF1 prefill: one long sequence cut into shards of whole blocks, one shard per rank (one
process per GPU, `torch.distributed`): contiguous ranges, or blocks dealt out round robin (`*_strided`).

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


def strided_blocks(n_tokens: int, rank: int, world: int) -> List[int]:
    """The blocks rank `rank` owns when blocks are dealt out round robin: rank, rank + world, ..."""
    nb = (n_tokens + BLOCK - 1) // BLOCK
    return list(range(rank, nb, world))


def exchange_plan_strided(n_tokens: int, world: int, cfg: Optional[B.RouteCfg] = None):
    """For every rank of a round-robin assignment the ascending list of blocks it reads but does not own."""
    plan = []
    for r in range(world):
        own = strided_blocks(n_tokens, r, world)
        plan.append(B.shard_needed_blocks_strided(n_tokens, r, world, len(own), cfg) if own else [])
    return plan


def exchange_blocks(k_local: torch.Tensor, v_local: torch.Tensor, owned: Sequence[Sequence[int]], rank: int,
                    needed: Sequence[Sequence[int]], group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Send this rank's blocks to the ranks that read them and receive the blocks this rank reads, for any
    assignment of blocks to ranks (`owned[r]`: ascending blocks of rank r; `needed[r]`: ascending blocks it is sent).

    k_local / v_local: this rank's own rows [own tokens, hkv, d], its blocks one after the other (only the last
    block of the sequence may be partial, and nobody reads it).  Returns the local "virtual sequence" tensors
    [len(needed[rank]) * 64 + own tokens, hkv, d]: the received blocks in ascending global order, then the own
    rows.  One message per (peer, tensor) in each direction; a peer's blocks that are consecutive in the needed
    list land directly in their place, scattered ones go through a receive buffer.
    """
    import torch.distributed as dist
    world = len(owned)
    owner = {p: r for r in range(world) for p in owned[r]}
    mine = list(needed[rank])
    place = {p: i for i, p in enumerate(mine)}
    my_index = {p: i for i, p in enumerate(owned[rank])}
    own_tokens = k_local.shape[0]
    out = []
    for t in (k_local, v_local):
        virt = torch.empty((len(mine) * BLOCK + own_tokens,) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        virt[len(mine) * BLOCK:] = t
        out.append(virt)
    ops, keep, scatter = [], [], []
    for src in range(world):
        blocks = [p for p in mine if owner[p] == src]
        if not blocks or src == rank:
            continue
        pos = [place[p] for p in blocks]
        direct = pos == list(range(pos[0], pos[0] + len(pos)))
        for virt in out:
            if direct:
                ops.append(dist.P2POp(dist.irecv, virt[pos[0] * BLOCK:(pos[0] + len(pos)) * BLOCK], src, group))
            else:
                buf = torch.empty((len(blocks) * BLOCK,) + tuple(virt.shape[1:]), dtype=virt.dtype, device=virt.device)
                scatter.append((virt, buf, pos))
                ops.append(dist.P2POp(dist.irecv, buf, src, group))
    for dst in range(world):
        if dst == rank:
            continue
        blocks = [p for p in needed[dst] if owner[p] == rank]
        if not blocks:
            continue
        rows = torch.cat([torch.arange(my_index[p] * BLOCK, (my_index[p] + 1) * BLOCK) for p in blocks]).to(k_local.device)
        for t in (k_local, v_local):
            buf = t.index_select(0, rows).contiguous()
            keep.append(buf)
            ops.append(dist.P2POp(dist.isend, buf, dst, group))
    if ops:
        for req in dist.batch_isend_irecv(ops):
            req.wait()
    for virt, buf, pos in scatter:
        rows = torch.cat([torch.arange(i * BLOCK, (i + 1) * BLOCK) for i in pos]).to(virt.device)
        virt.index_copy_(0, rows, buf)
    return out[0], out[1]


def exchange_kv(k_local: torch.Tensor, v_local: torch.Tensor, n_tokens: int, bounds: Sequence[int], rank: int,
                needed: Sequence[Sequence[int]], group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """`exchange_blocks` for contiguous shards (`bounds` from `shard_bounds`)."""
    owned = [list(range(bounds[r], bounds[r + 1])) for r in range(len(bounds) - 1)]
    return exchange_blocks(k_local, v_local, owned, rank, needed, group)


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


def shard_attn_fwd_strided(q_local, k_local, v_local, n_tokens: int, rank: int, world: int,
                           cfg: Optional[B.RouteCfg] = None, scale: Optional[float] = None, group=None):
    """The same with blocks dealt out round robin (rank r owns blocks r, r + world, ...): q_local / k_local / v_local
    hold the rank's blocks one after the other.  With a power-of-two `world` every rank is sent about two blocks per
    block of its own and all ranks carry the same work."""
    owned = [strided_blocks(n_tokens, r, world) for r in range(world)]
    needed = exchange_plan_strided(n_tokens, world, cfg)
    if not owned[rank]:
        return q_local[:0], torch.empty((q_local.shape[1], 0), dtype=torch.float32, device=q_local.device), 0
    k_virt, v_virt = exchange_blocks(k_local, v_local, owned, rank, needed, group)
    front = len(needed[rank]) * BLOCK
    q_virt = torch.zeros((front + q_local.shape[0],) + tuple(q_local.shape[1:]), dtype=q_local.dtype, device=q_local.device)
    q_virt[front:] = q_local
    nb = torch.tensor(needed[rank], dtype=torch.int32, device=q_local.device)
    route, cu = B.plan_route_shard_strided(n_tokens, rank, world, len(owned[rank]), nb, cfg)
    o, lse = B.attn_fwd(q_virt, k_virt, v_virt, cu, q_virt.shape[0], route, scale=scale)
    return o[front:], lse[:, front:], route
