"""CUDA attention path vs the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import bf1_inputs as I
import paper_2608_20427_b200 as bf1
from oracle import bf1_oracle as O

from gpu_util import assert_parity, errors, oracle_cfg, run_gpu

pytestmark = pytest.mark.gpu


def oracle_full(w, q, k, v, dense=False, scale=None, rows=None):
    if dense:
        return O.dense_causal(q, k, v, w.cu_seqlens(), scale=scale, rows=rows)
    return O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens(), scale=scale, rows=rows)


# the paper's gate lengths (Section 4.2: 128, 257, 512), block edges, and a one-token sequence
@pytest.mark.parametrize("n", [1, 2, 63, 64, 65, 128, 257, 512, 1000])
@pytest.mark.parametrize("d", [64, 128])
def test_small_lengths(n, d):
    w = I.custom([n], hq=4, hkv=2, d=d, seed=300 + n + d)
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v, guard=64)
    o_ref, lse_ref = oracle_full(w, q, k, v)
    assert_parity(o, lse, o_ref, lse_ref)


def test_config_tiny():
    w = I.WORKLOADS["tiny"]
    q, k, v = I.draw_qkv(w)
    o, lse, route = run_gpu(w, q, k, v, guard=64)
    o_ref, lse_ref = oracle_full(w, q, k, v)
    e = assert_parity(o, lse, o_ref, lse_ref)
    assert int(route.total_pairs.item()) == 270100
    print("tiny", e)


@pytest.mark.parametrize("dense", [False, True], ids=["bf1", "dense"])
def test_config_qwen_4k(dense):
    w = I.WORKLOADS["qwen_4k"]
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v, dense=dense)
    o_ref, lse_ref = oracle_full(w, q, k, v, dense=dense)
    print("qwen_4k", dense, assert_parity(o, lse, o_ref, lse_ref))


def test_dense_mode_small_and_equivalence_for_short_sequences():
    """Dense-path equivalence (Section 4.2): with every predecessor selected the operator is
    plain causal attention; for n <= 256 the BF1 route already selects every predecessor."""
    for n in (1, 64, 200, 256, 700):
        w = I.custom([n], hq=4, hkv=2, d=128, seed=400 + n)
        q, k, v = I.draw_qkv(w)
        o_d, lse_d, _ = run_gpu(w, q, k, v, dense=True, guard=64)
        o_ref, lse_ref = oracle_full(w, q, k, v, dense=True)
        assert_parity(o_d, lse_d, o_ref, lse_ref)
        if n <= 256:
            o_s, lse_s, _ = run_gpu(w, q, k, v)
            assert np.array_equal(o_s, o_d) and np.array_equal(lse_s, lse_d)


def test_ragged_small_batch_equals_per_sequence_launches_bitwise():
    lens = [130, 0, 257, 64, 1, 1000]
    w = I.custom(lens, hq=4, hkv=2, d=128, seed=500)
    q, k, v = I.draw_qkv(w)
    cu = w.cu_seqlens()
    for dense in (False, True):
        o, lse, _ = run_gpu(w, q, k, v, dense=dense, guard=64)
        o_ref, lse_ref = oracle_full(w, q, k, v, dense=dense)
        assert_parity(o, lse, o_ref, lse_ref)
        for s, n in enumerate(lens):
            if n == 0:
                continue
            sl = slice(cu[s], cu[s + 1])
            w1 = I.custom([n], hq=4, hkv=2, d=128, seed=0)
            o1, lse1, _ = run_gpu(w1, q[sl].contiguous(), k[sl].contiguous(), v[sl].contiguous(), dense=dense)
            assert np.array_equal(o[sl], o1) and np.array_equal(lse[:, sl], lse1)


def test_future_token_isolation_is_bitwise():
    """Section 4.2: zero output change under mutation of future tokens."""
    w = I.custom([600], hq=4, hkv=2, d=128, seed=600)
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v)
    for t in (0, 63, 64, 300, 598):
        q2, k2, v2 = I.mutate_after(w, q, k, v, 0, t, seed=700 + t)
        o2, lse2, _ = run_gpu(w, q2, k2, v2)
        assert np.array_equal(o[:t + 1], o2[:t + 1]) and np.array_equal(lse[:, :t + 1], lse2[:, :t + 1])
        assert not np.array_equal(o[t + 1:], o2[t + 1:])


@pytest.mark.parametrize("dense", [False, True], ids=["bf1", "dense"])
@pytest.mark.parametrize("hq,hkv", [(4, 2), (8, 2)], ids=["G2", "G4"])
def test_future_token_isolation_is_bitwise_when_later_rows_rescale(dense, hq, hkv):
    """The same gate on the path where it could fail: the kernel moves a row's reference maximum (and
    rescales its accumulator) only when that row's exponentials outgrow the guard, the whole warp then
    goes through the second pass together, and the rows of one warp are consecutive tokens.  The
    mutated tokens get Q and K rows 36x larger, so that they overflow in nearly every tile while the
    untouched rows never do; t sits in the middle of a 32-row group, so untouched and mutated rows
    share a warp.  Rows up to t must not change in a single bit."""
    n = 600
    w = I.custom([n], hq=hq, hkv=hkv, d=128, seed=650 + hq)
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v, dense=dense)
    for t in (305, 337 + 12, 46):          # positions 17, 29 and 14 of their 32-row groups
        q2, k2, v2 = I.mutate_after(w, q, k, v, 0, t, seed=750 + t, gain=36.0)
        o2, lse2, _ = run_gpu(w, q2, k2, v2, dense=dense)
        assert np.array_equal(o[:t + 1], o2[:t + 1]) and np.array_equal(lse[:, :t + 1], lse2[:, :t + 1])
        # the mutation did reach the later rows, and by the amounts the oracle predicts: their
        # scores are ~1300 times larger, so LSE moves by tens to thousands
        rows = np.arange(t + 1, n)
        o_ref, lse_ref = oracle_full(w, q2, k2, v2, dense=dense, rows=rows)
        assert np.abs(lse_ref[:, rows] - lse[:, rows]).min() > 10.0
        assert np.abs(lse2[:, rows] - lse_ref[:, rows]).max() <= 1e-3 * np.abs(lse_ref[:, rows]).max()
        diff = o2[rows].astype(np.float64) - o_ref[rows]
        assert np.sqrt((diff ** 2).mean() / (o_ref[rows].astype(np.float64) ** 2).mean()) <= 1e-2


def test_zero_queries_give_log_count():
    """Q = 0: every selected key gets the same weight, so LSE = ln(#selected columns)."""
    n = 1000
    w = I.custom([n], hq=2, hkv=1, d=64, seed=800)
    q, k, v = I.draw_qkv(w)
    q = torch.zeros_like(q)
    o, lse, _ = run_gpu(w, q, k, v)
    want = np.log(O.token_mask(O.cfg(), n).sum(axis=1).astype(np.float64))
    assert np.abs(lse[0] - want).max() < 1e-4
    assert np.abs(lse[1] - want).max() < 1e-4


def test_softmax_scale_argument():
    w = I.custom([300], hq=2, hkv=1, d=64, seed=900)
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v, scale=0.3)
    o_ref, lse_ref = oracle_full(w, q, k, v, scale=0.3)
    assert_parity(o, lse, o_ref, lse_ref)


def test_gqa_head_mapping_with_distinct_kv_heads():
    w = I.custom([320], hq=8, hkv=4, d=128, seed=1000)
    q, k, v = I.draw_qkv(w)
    o, lse, _ = run_gpu(w, q, k, v)
    o_ref, lse_ref = oracle_full(w, q, k, v)
    assert_parity(o, lse, o_ref, lse_ref)
    # per-head errors, so that a swapped head pair cannot hide in an average
    for h in range(8):
        assert np.abs(o[:, h] - o_ref[:, h]).max() <= 2e-2


def test_user_supplied_route_is_followed_and_bad_entries_are_flagged():
    """The kernel takes any ascending list ending in the query block (e.g. a sliding window)."""
    w = I.custom([1000], hq=2, hkv=1, d=64, seed=1100, local_blocks=4, global_first=0, dyadic=0)
    q, k, v = I.draw_qkv(w)
    o, lse, route = run_gpu(w, q, k, v)
    o_ref, lse_ref = oracle_full(w, q, k, v)
    assert_parity(o, lse, o_ref, lse_ref)
    # corrupt one list entry: out of range for its query block -> flagged, no fault
    dev = torch.device("cuda:0")
    route.kv_idx[3, 0] = 77
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
    bf1.attn_fwd(q.to(dev), k.to(dev), v.to(dev), cu, 1000, route)
    torch.cuda.synchronize()
    assert int(route.status.item()) & 8


@pytest.mark.parametrize("hq,hkv,d", [(4, 2, 128), (8, 2, 64)], ids=["G2-d128", "G4-d64"])
def test_static_random_route_written_by_hand(hq, hkv, d):
    """Section 4.3's static-random control: a route the planner did not write.  The test builds, on
    the host, a seeded random non-local block graph with the BF1 route's list lengths for two
    sequences (one with a partial last block), uploads it as a bf1_route and compares the kernel
    with the oracle's defining form under the boolean mask made from the very same lists."""
    from gpu_util import host_route, mask_from_lists
    lens = [4096, 1000]
    w = I.custom(lens, hq=hq, hkv=hkv, d=d, seed=1200 + d)
    q, k, v = I.draw_qkv(w)
    lists = [I.static_random_lists((n + 63) // 64, seed=17 + s) for s, n in enumerate(lens)]
    # the graph is non-local: most entries are neither the window, block 0 nor a dyadic predecessor
    bf1_sets = [set(np.flatnonzero(row)) for row in O.block_mask(O.cfg(), lens[0])]
    assert sum(len(set(lst) - bf1_sets[j]) for j, lst in enumerate(lists[0])) > 200
    arrays, total = host_route(lists, lens)
    dev = torch.device("cuda:0")
    route = bf1.Route.from_host(device=dev, total_pairs=total, **arrays)
    cu = bf1.cu_seqlens_tensor(lens, dev)
    T = w.total_tokens
    out = torch.full((T + 64, hq, d), float("nan"), dtype=torch.bfloat16, device=dev)
    lse = torch.full((hq, T), float("nan"), dtype=torch.float32, device=dev)
    bf1.attn_fwd(q.to(dev), k.to(dev), v.to(dev), cu, max(lens), route, out=out[:T], lse=lse)
    torch.cuda.synchronize()
    route.check_status()
    assert torch.isnan(out[T:].float()).all()
    o_gpu, lse_gpu = out[:T].float().cpu().numpy(), lse.cpu().numpy()
    cu_h = w.cu_seqlens()
    for s, n in enumerate(lens):
        sl = slice(cu_h[s], cu_h[s + 1])
        o_ref, lse_ref = O.attn_mask(q[sl], k[sl], v[sl], mask_from_lists(lists[s], n))
        assert_parity(o_gpu[sl], lse_gpu[:, sl], o_ref, lse_ref)
