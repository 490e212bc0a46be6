"""Shapes outside the five benchmark configurations: many short sequences, d = 64 at mid length,
a 128K-token sequence, other route topologies at full size (sampled rows)."""
import numpy as np
import pytest
import torch

import bf1_inputs as I
import paper_2608_20427_b200 as bf1
from oracle import bf1_oracle as O

from gpu_util import assert_parity, oracle_cfg, run_gpu
from test_gpu_full_size import sample_rows

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dense", [False, True], ids=["bf1", "dense"])
def test_batch_of_many_short_sequences(dense):
    rng = np.random.default_rng(5)
    lens = [int(x) for x in rng.integers(0, 300, size=400)]
    lens[7] = 0
    lens[8] = 64
    lens[9] = 1
    w = I.custom(lens, hq=4, hkv=2, d=128, seed=4000)
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v, dense=dense, guard=64)
    if dense:
        o_ref, lse_ref = O.dense_causal(q, k, v, w.cu_seqlens())
    else:
        o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens())
    assert_parity(o, lse, o_ref, lse_ref)


@pytest.mark.parametrize("dense", [False, True], ids=["bf1", "dense"])
def test_head_dim_64_mid_length(dense):
    w = I.custom([3001, 777], hq=8, hkv=4, d=64, seed=4100)
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v, dense=dense, guard=64)
    rows = sample_rows(w, per_seq=120)
    if dense:
        o_ref, lse_ref = O.dense_causal(q, k, v, w.cu_seqlens(), rows=rows)
    else:
        o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens(), rows=rows)
    assert_parity(o, lse, o_ref, lse_ref, rows=rows)


def test_128k_tokens():
    w = I.custom([131072], hq=2, hkv=1, d=128, seed=4200)
    q, k, v = I.draw_qkv(w)
    o, lse, route = run_gpu(w, q, k, v)
    assert route.max_degree == 13 and int(route.num_qblocks.item()) == 2048
    rows = sample_rows(w, per_seq=150)
    o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens(), rows=rows)
    assert_parity(o, lse, o_ref, lse_ref, rows=rows)


@pytest.mark.parametrize("route", [dict(local_blocks=9, global_first=0, dyadic=0),     # sliding window
                                   dict(local_blocks=0, global_first=1, dyadic=1),     # no local window
                                   dict(local_blocks=40, global_first=1, dyadic=1)],   # lists longer than a warp
                         ids=["sliding", "dyadic-only", "wide"])
def test_other_routes_at_16k(route):
    w = I.custom([16384], hq=4, hkv=2, d=128, seed=4300, **route)
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v)
    rows = sample_rows(w, per_seq=120)
    o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens(), rows=rows)
    assert_parity(o, lse, o_ref, lse_ref, rows=rows)


@pytest.mark.parametrize("q_gain,k_top", [(3.0, 6.0), (6.0, 12.0), (12.0, 40.0)], ids=["lagging", "guard", "overflow"])
def test_large_scores_do_not_break_the_lazy_reference(q_gain, k_top):
    """The kernel takes a tile's exponentials against the row's reference maximum of earlier tiles and
    only moves the reference when the tile's row sum reaches 2^60 (or overflows).  Scores that grow tile
    after tile exercise the three regimes: the reference lags by tens of binary orders and is never
    moved, the sum trips the guard while still finite, the exponentials overflow outright.  The result
    must match the oracle in all of them."""
    w = I.custom([1024], hq=2, hkv=1, d=64, seed=4400)
    q, k, v = I.draw_qkv(w)
    ramp = torch.linspace(0.2, k_top, 1024).reshape(-1, 1, 1)
    k = (k.float() * ramp).to(torch.bfloat16)           # later keys score much higher
    q = (q.float() * q_gain).to(torch.bfloat16)
    for dense in (False, True):
        o, lse, _ = run_gpu(w, q, k, v, dense=dense)
        if dense:
            o_ref, lse_ref = O.dense_causal(q, k, v, w.cu_seqlens())
        else:
            o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens())
        assert not np.isnan(o).any()
        # LSE is large here (hundreds to thousands): compare relative to its size
        assert np.abs(lse - lse_ref).max() <= 1e-3 * max(1.0, np.abs(lse_ref).max())
        diff = o.astype(np.float64) - o_ref
        assert np.abs(diff).max() <= 4e-2 and np.sqrt((diff ** 2).mean() / (o_ref.astype(np.float64) ** 2).mean()) <= 1e-2


@pytest.mark.parametrize("dense", [False, True], ids=["bf1", "dense"])
@pytest.mark.parametrize("d", [64, 128])
def test_group_of_four_query_heads(dense, d):
    """G = 4 (e.g. 32 query / 8 KV heads): the tile is 4 heads x 32 tokens, a query block is two units."""
    w = I.custom([1, 31, 32, 33, 64, 97, 1000, 2500], hq=8, hkv=2, d=d, seed=4500 + d)
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v, dense=dense, guard=64)
    if dense:
        o_ref, lse_ref = O.dense_causal(q, k, v, w.cu_seqlens())
    else:
        o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens())
    assert_parity(o, lse, o_ref, lse_ref)
    for h in range(8):   # per head, so that a permuted head cannot hide in an average
        assert np.abs(o[:, h] - o_ref[:, h]).max() <= 2e-2


@pytest.mark.parametrize("dense", [False, True], ids=["bf1", "dense"])
@pytest.mark.parametrize("d", [64, 128])
def test_one_query_head_per_kv_head(dense, d):
    """G = 1 (plain multi-head attention): one head fills rows 0..63 of the 128-row tile, the other half is idle."""
    w = I.custom([1, 63, 64, 65, 257, 1000, 2500], hq=3, hkv=3, d=d, seed=4600 + d)
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v, dense=dense, guard=64)
    if dense:
        o_ref, lse_ref = O.dense_causal(q, k, v, w.cu_seqlens())
    else:
        o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens())
    assert_parity(o, lse, o_ref, lse_ref)
    for h in range(3):
        assert np.abs(o[:, h] - o_ref[:, h]).max() <= 2e-2
