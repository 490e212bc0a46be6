"""Route block width b = 128 through planner, forward, backward and decode.

The kernels work on 64-token tiles; at b = 128 the planner writes, for every tile, the tiles of the
blocks Eq. 1 selects for the tile's 128-token block.  The oracle is run with block = 128 and knows
nothing of tiles: masks and totals must agree bit for bit, outputs and gradients within the usual
tolerances."""
import numpy as np
import pytest
import torch

import bf1_inputs as I
import paper_2608_20427_b200 as bf1
from oracle import bf1_oracle as O

from gpu_util import assert_parity, lib_cfg, mask_from_lists, oracle_cfg, run_gpu
from test_gpu_decode import paged_cache, run_decode
from test_gpu_backward import REL_MAX, REL_RMS, run_case

pytestmark = pytest.mark.gpu

ROUTES = [dict(), dict(local_blocks=0), dict(local_blocks=3, global_first=0, dyadic=0), dict(global_first=0)]


@pytest.mark.parametrize("n", [1, 64, 65, 128, 129, 257, 1000, 4096, 5000])
@pytest.mark.parametrize("kw", ROUTES, ids=lambda k: ",".join("%s=%s" % i for i in k.items()) or "paper")
def test_tile_lists_select_the_token_mask_of_the_wider_block(n, kw):
    dev = torch.device("cuda:0")
    cu = bf1.cu_seqlens_tensor([n], dev)
    route = bf1.plan_route(cu, n, bf1.RouteCfg(block=128, **kw))
    torch.cuda.synchronize()
    route.check_status()
    tiles = (n + 63) // 64
    assert int(route.num_qblocks.item()) == tiles
    assert route.qb_block[:tiles].tolist() == list(range(tiles))
    cnt = route.kv_count[:tiles].cpu().numpy()
    idx = route.kv_idx[:tiles].cpu().numpy()
    lists = [idx[t, :cnt[t]].tolist() for t in range(tiles)]
    for t, lst in enumerate(lists):
        assert lst == sorted(set(lst)) and lst[-1] == t and (idx[t, cnt[t]:] == -1).all()
    c = O.cfg(block=128, **kw)
    assert (mask_from_lists(lists, n, block=64) == O.token_mask(c, n)).all()
    # totals: the oracle counts per 128-token block, the planner per tile
    _, _, pairs, total = O.route(c, n)
    assert int(route.total_pairs.item()) == int(total) == int(np.asarray(pairs).sum())
    got = route.pair_count[:tiles].cpu().numpy().astype(np.int64)
    per_block = np.add.reduceat(got, np.arange(0, tiles, 2))
    assert np.array_equal(per_block, np.asarray(pairs, dtype=np.int64))
    # capacity helper: tiles, and twice the block-level list length
    cap, deg = bf1.route_capacity(1, n, n, bf1.RouteCfg(block=128, **kw))
    assert cap >= tiles and deg == route.max_degree and cnt.max() <= deg
    if n >= 4096 and not kw:
        assert cnt.max() == deg


@pytest.mark.parametrize("lens,hq,hkv,d", [([1000], 4, 2, 128), ([130, 0, 257, 64, 1, 700], 4, 2, 64),
                                           ([3001], 8, 2, 128), ([2000], 3, 3, 64)],
                         ids=["G2-d128", "ragged-d64", "G4-d128", "G1-d64"])
def test_forward_matches_the_oracle_at_b128(lens, hq, hkv, d):
    w = I.custom(lens, hq=hq, hkv=hkv, d=d, seed=12800 + sum(lens), block=128)
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v, guard=64)
    o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens())
    print(assert_parity(o, lse, o_ref, lse_ref))


def test_forward_16k_at_b128_sampled_rows():
    w = I.custom([16384], hq=16, hkv=8, d=128, seed=12816, block=128)
    q, k, v = I.draw_qkv(w)
    o, lse, route = run_gpu(w, q, k, v)
    rows = list(range(0, 16384, 97)) + [16383, 16320, 127, 128]
    o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens(), rows=rows)
    assert_parity(o, lse, o_ref, lse_ref, rows=rows)
    assert int(route.total_pairs.item()) == int(O.route(oracle_cfg(w), 16384)[3])


def test_backward_matches_the_oracle_at_b128():
    w = I.custom([1000, 257], hq=4, hkv=2, d=128, seed=12830, block=128)
    res = run_case(w, seed=3)
    print(res)
    for name, (rms, mx) in res.items():
        assert rms <= REL_RMS and mx <= REL_MAX, (name, rms, mx)


@pytest.mark.parametrize("lens", [[1, 64, 65, 128, 129, 193, 1000, 0, 4097], [700] * 40], ids=["tails", "many"])
def test_decode_matches_the_oracle_at_b128(lens):
    w = I.custom(lens, hq=4, hkv=2, d=128, seed=12840, block=128)
    q, k, v = I.draw_qkv(w)
    kp, vp, table = paged_cache(w, k, v, seed=5)
    dev = torch.device("cuda:0")
    sl = torch.tensor(list(w.seqlens), dtype=torch.int32, device=dev)
    plan = bf1.plan_decode(sl, table.to(dev), lib_cfg(w))
    out, lse, plan, last = run_decode(w, q, kp, vp, table, plan=plan)
    assert int(plan.status.item()) == 0
    rows = [r for r, n in zip(last, w.seqlens) if n > 0]
    live = [s for s, n in enumerate(w.seqlens) if n > 0]
    o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens(), rows=rows)
    assert_parity(out[live], lse[:, live], o_ref[rows], lse_ref[:, rows])


def test_sequence_sharding_refuses_b128():
    with pytest.raises(bf1.Bf1Error):
        bf1.shard_needed_blocks(4096, 0, 8, bf1.RouteCfg(block=128))
