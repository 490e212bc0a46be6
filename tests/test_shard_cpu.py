"""Sequence-sharded prefill, the parts that need no GPU: which blocks a shard must be sent (against the oracle's
block mask), and the exchange itself between two and three `gloo` ranks on CPU tensors -- after it, every rank
holds a local key/value tensor on which the oracle, under the mask of the re-indexed lists, reproduces the rows of
the full-sequence oracle bit for bit."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bf1_inputs as I
import paper_2608_20427_b200 as bf1
from paper_2608_20427_b200 import shard
from oracle import bf1_oracle as O


def oracle_needed(cfg, n, lo, hi):
    bm = O.block_mask(cfg, n)
    return [p for p in range(lo) if bm[lo:hi, p].any()]


@pytest.mark.parametrize("route", [dict(), dict(local_blocks=5, global_first=0, dyadic=0), dict(local_blocks=0)],
                         ids=["bf1", "sliding", "no-window"])
def test_needed_blocks_match_the_oracle_block_mask(route):
    rng = np.random.default_rng(11)
    w = I.custom([1], 2, 1, 64, seed=0, **route)
    ocfg = O.cfg(w.block, w.local_blocks, w.global_first, w.dyadic)
    lcfg = bf1.RouteCfg(w.block, w.local_blocks, w.global_first, w.dyadic)
    for n in (1, 64, 65, 1000, 4097, 20000):
        nb = (n + 63) // 64
        for _ in range(6):
            lo = int(rng.integers(0, nb))
            hi = int(rng.integers(lo + 1, nb + 1))
            assert bf1.shard_needed_blocks(n, lo, hi, lcfg) == oracle_needed(ocfg, n, lo, hi), (n, lo, hi)
    # a shard that starts at block 0 needs nothing; bad ranges are refused
    assert bf1.shard_needed_blocks(1000, 0, 16, lcfg) == []
    with pytest.raises(bf1.Bf1Error):
        bf1.shard_needed_blocks(1000, 3, 3, lcfg)
    with pytest.raises(bf1.Bf1Error):
        bf1.shard_needed_blocks(1000, 3, 17, lcfg)


def test_contiguous_shards_of_the_dyadic_route_need_most_of_what_lies_in_front_of_them():
    """The dyadic offsets of 128 consecutive query blocks sweep whole ranges: at 32K with four shards the
    last rank reads 257 of the 384 blocks in front of it (Proposition 1 bounds the blocks per QUERY block, not
    per shard); the exchange is static, not small."""
    plan = shard.exchange_plan(32768, shard.shard_bounds(32768, 4))
    assert [len(x) for x in plan] == [0, 128, 256, 257]


def test_strided_shards_are_balanced_and_match_the_oracle_block_mask():
    """Blocks dealt out round robin: a rank is sent the selected blocks it does not own.  With four ranks at 32K
    every rank is sent 254 to 257 blocks (contiguous shards: 0, 128, 256, 257) and holds lists of the same lengths,
    because the dyadic predecessors j - 2^k, 2^k >= 4, of an owned block are owned too."""
    assert [len(x) for x in shard.exchange_plan_strided(32768, 4)] == [254, 255, 256, 257]
    cfg = O.cfg()
    for n, world in ((1000, 2), (4097, 3), (20000, 8), (64, 4)):
        bm = O.block_mask(cfg, n)
        nb = bm.shape[0]
        plan = shard.exchange_plan_strided(n, world)
        for r in range(world):
            own = shard.strided_blocks(n, r, world)
            want = sorted({p for j in own for p in np.nonzero(bm[j])[0] if p % world != r})
            assert plan[r] == want, (n, world, r)
        assert sorted(p for r in range(world) for p in shard.strided_blocks(n, r, world)) == list(range(nb))
    with pytest.raises(bf1.Bf1Error):
        bf1.shard_needed_blocks_strided(1000, 3, 4, 5)       # block 19 does not exist
    with pytest.raises(bf1.Bf1Error):
        bf1.shard_needed_blocks_strided(1000, 0, 0, 4)


def _rank_main(rank, world, port, n, seed, out, strided=False):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = I.custom([n], hq=2, hkv=1, d=64, seed=seed)
    q, k, v = I.draw_qkv(w)                        # every rank draws the same sequence and keeps its shard
    if strided:
        owned = [shard.strided_blocks(n, r, world) for r in range(world)]
        needed = shard.exchange_plan_strided(n, world)
    else:
        bounds = shard.shard_bounds(n, world)
        owned = [list(range(bounds[r], bounds[r + 1])) for r in range(world)]
        needed = shard.exchange_plan(n, bounds)
    own = owned[rank]
    own_rows = torch.cat([torch.arange(j * 64, min(j * 64 + 64, n)) for j in own]).long()
    k_virt, v_virt = shard.exchange_blocks(k[own_rows].contiguous(), v[own_rows].contiguous(), owned, rank, needed)
    # what arrived is what the plan names, in that order
    rows = torch.cat([torch.arange(p * 64, p * 64 + 64) for p in needed[rank]] + [own_rows]).long()
    ok_data = bool(torch.equal(k_virt, k[rows]) and torch.equal(v_virt, v[rows]))
    # the oracle on the local tensor, under the mask of the re-indexed lists, equals the full-sequence oracle
    cfg = O.cfg()
    idx, cnt, _, _ = O.route(cfg, n)
    front = len(needed[rank])
    nv = front * 64 + len(own_rows)
    lists = [[] for _ in range(front)]             # the landing blocks have no query rows: empty lists
    place = {p: i for i, p in enumerate(needed[rank])}
    mine = {p: front + i for i, p in enumerate(own)}
    for j in own:
        lists.append([mine[p] if p in mine else place[p] for p in idx[j, :cnt[j]]])
    mask = np.zeros((nv, nv), dtype=bool)
    for jj, lst in enumerate(lists):
        r0, r1 = jj * 64, min(jj * 64 + 64, nv)
        for p in lst:
            mask[r0:r1, p * 64:min(p * 64 + 64, nv)] = True
    # causal triangle inside the self block only: every other listed block lies wholly in the past, wherever the
    # local numbering puts it
    for g in range(len(own)):
        r0, r1 = (front + g) * 64, min((front + g) * 64 + 64, nv)
        blk = mask[r0:r1, r0:r1]
        mask[r0:r1, r0:r1] = blk & np.tril(np.ones(blk.shape, dtype=bool))
    mask[:front * 64, 0] = True                    # rows without a query still need one column for the oracle
    q_virt = torch.zeros((nv, 2, 64), dtype=torch.bfloat16)
    q_virt[front * 64:] = q[own_rows]
    own_np = own_rows.numpy()
    if not strided:
        # the local tensor keeps the keys in their global order: the oracle adds in the same order, bit for bit
        o_loc, lse_loc = O.attn_mask(q_virt, k_virt, v_virt, mask)
        o_full, lse_full = O.attn_route(cfg, q, k, v, [0, n], rows=own_rows.tolist())
        ok_attn = bool(np.array_equal(o_loc[front * 64:], o_full[own_np]) and np.array_equal(lse_loc[:, front * 64:], lse_full[:, own_np]))
    else:
        # round robin puts the received blocks in front of the own ones, so the sums run in another order:
        # compare in fp64, where the order costs 1e-15
        o_loc, lse_loc = O.attn_mask(q_virt, k_virt, v_virt, mask, fp64=True)
        o_full, lse_full = O.attn_route(cfg, q, k, v, [0, n], rows=own_rows.tolist(), fp64=True)
        ok_attn = bool(np.abs(o_loc[front * 64:] - o_full[own_np]).max() < 1e-12 and
                       np.abs(lse_loc[:, front * 64:] - lse_full[:, own_np]).max() < 1e-12)
    gathered = [None] * world
    dist.all_gather_object(gathered, (ok_data, ok_attn, len(needed[rank])))
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,n,strided", [(2, 1000, False), (3, 2500, False), (2, 1000, True), (4, 2500, True)],
                         ids=["contiguous-2", "contiguous-3", "strided-2", "strided-4"])
def test_exchange_between_gloo_ranks(world, n, strided):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29700 + (os.getpid() + world + 7 * strided) % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, n, 8100 + n, out, strided)) for r in range(world)]
    for p in procs:
        p.start()
    res = out.get(timeout=300)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert all(ok_data and ok_attn for ok_data, ok_attn, _ in res), res
    assert (res[0][2] == 0 or strided) and all(c > 0 for _, _, c in res[1:])
