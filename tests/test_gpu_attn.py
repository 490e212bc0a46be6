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
