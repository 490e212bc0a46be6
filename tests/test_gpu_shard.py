"""Sequence-sharded prefill on one GPU: the shards of a sequence are run one after another (what each rank of a
multi-GPU job would do after its exchange), each on its own local [received | own] key/value tensor through the route
that bf1_plan_route_shard re-indexes on the device.  The lists must equal the oracle's lists in the local numbering,
the pair totals must add up to the sequence's, and O / LSE must equal the unsharded launch bit for bit."""
import numpy as np
import pytest
import torch

import bf1_inputs as I
import paper_2608_20427_b200 as bf1
from paper_2608_20427_b200 import shard
from oracle import bf1_oracle as O

from gpu_util import assert_parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,world,hq,hkv,d", [(1000, 2, 4, 2, 128), (4097, 3, 4, 2, 64), (16384, 4, 16, 8, 128)])
def test_shards_reproduce_the_unsharded_launch(n, world, hq, hkv, d):
    dev = torch.device("cuda:0")
    w = I.custom([n], hq=hq, hkv=hkv, d=d, seed=9000 + n)
    q, k, v = I.draw_qkv(w)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    cu = bf1.cu_seqlens_tensor([n], dev)
    full = bf1.plan_route(cu, n)
    o_full, lse_full = bf1.attn_fwd(qd, kd, vd, cu, n, full)
    torch.cuda.synchronize()
    full.check_status()
    idx, cnt, pairs, total = O.route(O.cfg(), n, full.max_degree)
    bounds = shard.shard_bounds(n, world)
    needed = shard.exchange_plan(n, bounds)
    got_pairs = 0
    for rank in range(world):
        lo, hi = bounds[rank], bounds[rank + 1]
        t0, t1 = lo * 64, min(hi * 64, n)
        front = len(needed[rank])
        rows = torch.cat([torch.arange(p * 64, p * 64 + 64) for p in needed[rank]] + [torch.arange(t0, t1)]).to(dev)
        k_virt, v_virt = kd[rows].contiguous(), vd[rows].contiguous()     # stands in for the exchange
        q_virt = torch.zeros((front * 64 + t1 - t0, hq, d), dtype=torch.bfloat16, device=dev)
        q_virt[front * 64:] = qd[t0:t1]
        route, cu_s = bf1.plan_route_shard(n, lo, hi, torch.tensor(needed[rank], dtype=torch.int32, device=dev))
        torch.cuda.synchronize()
        route.check_status()
        assert cu_s.tolist() == [0, front * 64 + t1 - t0]
        # the device's re-indexed lists against the oracle's, mapped by hand
        place = {p: i for i, p in enumerate(needed[rank])}
        want = np.full((hi - lo, route.max_degree), -1, dtype=np.int32)
        for j in range(lo, hi):
            want[j - lo, :cnt[j]] = [place[p] if p < lo else front + (p - lo) for p in idx[j, :cnt[j]]]
        assert np.array_equal(route.kv_idx[:hi - lo].cpu().numpy(), want)
        assert np.array_equal(route.kv_count[:hi - lo].cpu().numpy(), cnt[lo:hi])
        assert np.array_equal(route.qb_block[:hi - lo].cpu().numpy(), front + np.arange(hi - lo))
        assert np.array_equal(route.pair_count[:hi - lo].cpu().numpy(), pairs[lo:hi])
        assert sorted(route.order[:hi - lo].cpu().tolist()) == list(range(hi - lo))
        got_pairs += int(route.total_pairs.item())
        o = torch.full(q_virt.shape, float("nan"), dtype=torch.bfloat16, device=dev)
        lse = torch.full((hq, q_virt.shape[0]), float("nan"), dtype=torch.float32, device=dev)
        bf1.attn_fwd(q_virt, k_virt, v_virt, cu_s, q_virt.shape[0], route, out=o, lse=lse)
        torch.cuda.synchronize()
        route.check_status()
        assert torch.equal(o[front * 64:], o_full[t0:t1]) and torch.equal(lse[:, front * 64:], lse_full[:, t0:t1])
        assert torch.isnan(o[:front * 64].float()).all()            # the landing rows have no queries: never written
    assert got_pairs == total == int(full.total_pairs.item())
    # and the unsharded launch itself is the oracle's answer (sampled rows at the larger sizes)
    rows = np.unique(np.concatenate([np.arange(0, n, max(1, n // 300)), [n - 1]]))
    o_ref, lse_ref = O.attn_route(O.cfg(), q, k, v, [0, n], rows=rows)
    assert_parity(o_full.float().cpu().numpy(), lse_full.cpu().numpy(), o_ref, lse_ref, rows=rows)


@pytest.mark.parametrize("n,world,hq,hkv,d", [(1000, 2, 4, 2, 128), (4097, 3, 4, 2, 64), (16384, 4, 16, 8, 128), (64, 4, 2, 1, 64)])
def test_round_robin_shards_reproduce_the_unsharded_launch(n, world, hq, hkv, d):
    """Blocks dealt out round robin (rank r owns r, r + world, ...).  Lists are re-indexed entry by entry, so the
    kernel walks a query block's tiles in the same order as the unsharded launch: O and LSE must be bit-identical."""
    dev = torch.device("cuda:0")
    w = I.custom([n], hq=hq, hkv=hkv, d=d, seed=9100 + n)
    q, k, v = I.draw_qkv(w)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    cu = bf1.cu_seqlens_tensor([n], dev)
    full = bf1.plan_route(cu, n)
    o_full, lse_full = bf1.attn_fwd(qd, kd, vd, cu, n, full)
    torch.cuda.synchronize()
    full.check_status()
    idx, cnt, pairs, total = O.route(O.cfg(), n, full.max_degree)
    needed = shard.exchange_plan_strided(n, world)
    got_pairs = 0
    for rank in range(world):
        own = shard.strided_blocks(n, rank, world)
        if not own:
            assert needed[rank] == []
            continue
        own_rows = torch.cat([torch.arange(j * 64, min(j * 64 + 64, n)) for j in own]).to(dev)
        front = len(needed[rank])
        rows = torch.cat([torch.arange(p * 64, p * 64 + 64) for p in needed[rank]] + [own_rows.cpu()]).to(dev)
        k_virt, v_virt = kd[rows].contiguous(), vd[rows].contiguous()     # stands in for the exchange
        q_virt = torch.zeros((front * 64 + own_rows.numel(), hq, d), dtype=torch.bfloat16, device=dev)
        q_virt[front * 64:] = qd[own_rows]
        route, cu_s = bf1.plan_route_shard_strided(n, rank, world, len(own), torch.tensor(needed[rank], dtype=torch.int32, device=dev))
        torch.cuda.synchronize()
        route.check_status()
        assert cu_s.tolist() == [0, front * 64 + own_rows.numel()]
        place = {p: i for i, p in enumerate(needed[rank])}
        mine = {p: front + i for i, p in enumerate(own)}
        want = np.full((len(own), route.max_degree), -1, dtype=np.int32)
        for g, j in enumerate(own):
            want[g, :cnt[j]] = [mine[p] if p in mine else place[p] for p in idx[j, :cnt[j]]]
        assert np.array_equal(route.kv_idx[:len(own)].cpu().numpy(), want)
        assert np.array_equal(route.kv_count[:len(own)].cpu().numpy(), cnt[own])
        assert np.array_equal(route.qb_block[:len(own)].cpu().numpy(), front + np.arange(len(own)))
        assert np.array_equal(route.pair_count[:len(own)].cpu().numpy(), pairs[own])
        got_pairs += int(route.total_pairs.item())
        o = torch.full(q_virt.shape, float("nan"), dtype=torch.bfloat16, device=dev)
        lse = torch.full((hq, q_virt.shape[0]), float("nan"), dtype=torch.float32, device=dev)
        bf1.attn_fwd(q_virt, k_virt, v_virt, cu_s, q_virt.shape[0], route, out=o, lse=lse)
        torch.cuda.synchronize()
        route.check_status()
        assert torch.equal(o[front * 64:], o_full[own_rows]) and torch.equal(lse[:, front * 64:], lse_full[:, own_rows])
        assert torch.isnan(o[:front * 64].float()).all()
    assert got_pairs == total == int(full.total_pairs.item())


def test_a_block_missing_from_the_landing_list_is_flagged():
    dev = torch.device("cuda:0")
    needed = bf1.shard_needed_blocks(4096, 32, 64)
    route, _ = bf1.plan_route_shard(4096, 32, 64, torch.tensor(needed[:-1], dtype=torch.int32, device=dev))
    torch.cuda.synchronize()
    assert int(route.status.item()) & 8 and int(route.num_qblocks.item()) == 0
