"""Device route planner vs the oracle: lists, lengths and pair counts must match bit for bit."""
import numpy as np
import pytest
import torch

import bf1_inputs as I
import paper_2608_20427_b200 as bf1
from oracle import bf1_oracle as O

pytestmark = pytest.mark.gpu

CASES = [
    [1], [63], [64], [65], [128], [257], [512], [1000], [2048], [4096], [8192], [16384], [32768],
    [3001, 8192, 12345, 16384], [130, 0, 257, 64, 1], [0, 0, 5], [70000],
]
CFGS = [dict(), dict(local_blocks=0), dict(local_blocks=5, global_first=0, dyadic=0),
        dict(global_first=0), dict(local_blocks=1, dyadic=0)]


def oracle_route(seqlens, kw, max_deg):
    c = O.cfg(**kw)
    seq, blk, cnt, idx, pairs = [], [], [], [], []
    for s, n in enumerate(seqlens):
        if n == 0:
            continue
        i, c_, p, _ = O.route(c, n, max_deg)
        B = len(c_)
        seq += [s] * B
        blk += list(range(B))
        cnt.append(c_)
        idx.append(i)
        pairs.append(p)
    if not cnt:
        return (np.zeros(0, np.int32),) * 3 + (np.zeros((0, max_deg), np.int32), np.zeros(0, np.int64))
    return (np.array(seq, np.int32), np.array(blk, np.int32), np.concatenate(cnt), np.concatenate(idx),
            np.concatenate(pairs))


@pytest.mark.parametrize("seqlens", CASES, ids=lambda s: "-".join(map(str, s)))
@pytest.mark.parametrize("kw", CFGS, ids=lambda k: ",".join("%s=%s" % i for i in k.items()) or "paper")
def test_planner_matches_oracle_bit_exact(seqlens, kw):
    dev = torch.device("cuda:0")
    cu = bf1.cu_seqlens_tensor(seqlens, dev)
    route = bf1.plan_route(cu, max(seqlens), bf1.RouteCfg(**kw))
    torch.cuda.synchronize()
    route.check_status()
    nqb = int(route.num_qblocks.item())
    seq, blk, cnt, idx, pairs = oracle_route(seqlens, kw, route.max_degree)
    assert nqb == len(seq)
    assert np.array_equal(route.qb_seq[:nqb].cpu().numpy(), seq)
    assert np.array_equal(route.qb_block[:nqb].cpu().numpy(), blk)
    assert np.array_equal(route.kv_count[:nqb].cpu().numpy(), cnt)
    assert np.array_equal(route.kv_idx[:nqb].cpu().numpy(), idx)
    assert np.array_equal(route.pair_count[:nqb].cpu().numpy().astype(np.int64), pairs)
    assert int(route.total_pairs.item()) == int(pairs.sum())
    # hand-out order: a permutation of the slots with non-increasing list length
    order = route.order[:nqb].cpu().numpy()
    assert np.array_equal(np.sort(order), np.arange(nqb))
    assert (np.diff(cnt[order]) <= 0).all()


def test_planner_flags_bad_sequence_lengths_without_faulting():
    dev = torch.device("cuda:0")
    cu = torch.tensor([0, 100, 90, 300], dtype=torch.int32, device=dev)   # decreasing
    cap, deg = bf1.route_capacity(3, 300, 300)
    route = bf1.Route.empty(cap, deg, dev)
    cu._bf1_total = 300
    bf1.plan_route(cu, 300, route=route)
    torch.cuda.synchronize()
    assert int(route.status.item()) & 1 and int(route.num_qblocks.item()) == 0
    # a sequence longer than max_seqlen
    cu = bf1.cu_seqlens_tensor([100, 200], dev)
    route = bf1.Route.empty(cap, deg, dev)
    bf1.plan_route(cu, 150, route=route)
    torch.cuda.synchronize()
    assert int(route.status.item()) & 1
    # too few slots
    cu = bf1.cu_seqlens_tensor([1000], dev)
    route = bf1.Route.empty(4, 6, dev)
    bf1.plan_route(cu, 1000, route=route)
    torch.cuda.synchronize()
    assert int(route.status.item()) & 2 and int(route.num_qblocks.item()) == 0
    # list pitch too small is caught on the host
    route = bf1.Route.empty(16, 3, dev)
    with pytest.raises(bf1.Bf1Error):
        bf1.plan_route(cu, 1000, route=route)
    # and a good plan afterwards clears the status word
    route = bf1.plan_route(cu, 1000)
    torch.cuda.synchronize()
    assert int(route.status.item()) == 0 and int(route.num_qblocks.item()) == 16
