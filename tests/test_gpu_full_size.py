"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (one plan
reused by back-to-back bf1_attn_fwd calls), on sampled output rows the oracle computes one by one."""
import numpy as np
import pytest
import torch

import bf1_inputs as I
import paper_2608_20427_b200 as bf1
from oracle import bf1_oracle as O

from gpu_util import assert_parity, oracle_cfg

pytestmark = pytest.mark.gpu


def sample_rows(w, per_seq=160, seed=0):
    """Global token rows: block edges, first / last rows of every sequence, and a random spread."""
    rng = np.random.default_rng(seed)
    rows = set()
    cu = w.cu_seqlens()
    for s, n in enumerate(w.seqlens):
        if n == 0:
            continue
        local = {0, n - 1, min(63, n - 1), min(64, n - 1), n // 2, (n // 64) * 64 if n % 64 else n - 64,
                 max(n - 2, 0), min(255, n - 1), min(256, n - 1), min(4095, n - 1), min(4096, n - 1)}
        local |= set(int(x) for x in rng.integers(0, n, size=per_seq))
        # one full block in the middle, so that a whole tile's rows are checked together
        mid = (n // 128) * 64
        local |= set(range(mid, min(mid + 64, n)))
        rows |= {cu[s] + r for r in local if 0 <= r < n}
    return np.array(sorted(rows), dtype=np.int64)


def gpu_layers(w, layers, dense=False):
    """Plan once, then `layers` back-to-back calls on independent inputs (what bench.py times)."""
    dev = torch.device("cuda:0")
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
    T = w.total_tokens
    route = None if dense else bf1.plan_route(cu, w.max_seqlen)
    work = torch.zeros(4, dtype=torch.int32, device=dev)
    inputs = [I.draw_qkv(w, layer=layer) for layer in range(layers)]
    dev_in = [tuple(t.to(dev) for t in x) for x in inputs]
    outs = [torch.full((T, w.hq, w.d), float("nan"), dtype=torch.bfloat16, device=dev) for _ in range(layers)]
    lses = [torch.full((w.hq, T), float("nan"), dtype=torch.float32, device=dev) for _ in range(layers)]
    for layer in range(layers):
        q, k, v = dev_in[layer]
        if dense:
            bf1.dense_causal_fwd(q, k, v, cu, w.max_seqlen, out=outs[layer], lse=lses[layer], work=work)
        else:
            bf1.attn_fwd(q, k, v, cu, w.max_seqlen, route, out=outs[layer], lse=lses[layer])
    torch.cuda.synchronize()
    if dense:
        assert work.tolist() == [0, 0, 0, 0]
    else:
        route.check_status()
    return inputs, [o.float().cpu().numpy() for o in outs], [x.cpu().numpy() for x in lses], route


def check(w, inputs, outs, lses, rows, dense=False):
    worst = {}
    for (q, k, v), o, lse in zip(inputs, outs, lses):
        assert not np.isnan(o).any() and not np.isnan(lse).any(), "unwritten output rows"
        if dense:
            o_ref, lse_ref = O.dense_causal(q, k, v, w.cu_seqlens(), rows=rows)
        else:
            o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens(), rows=rows)
        e = assert_parity(o, lse, o_ref, lse_ref, rows=rows)
        for key, val in e.items():
            worst[key] = max(worst.get(key, 0.0), val)
    return worst


def test_long_context_32k_eight_layers_share_one_plan():
    w = I.WORKLOADS["qwen_32k"]
    inputs, outs, lses, route = gpu_layers(w, 8)
    assert int(route.total_pairs.item()) == 19_902_464
    rows = sample_rows(w, per_seq=200)
    print("32k x 8 layers", check(w, inputs, outs, lses, rows))


@pytest.mark.parametrize("name", ["qwen_2k", "qwen_8k", "qwen_16k"])
def test_length_sweep_bf1_and_dense(name):
    w = I.WORKLOADS[name]
    n = w.seqlens[0]
    inputs, outs, lses, route = gpu_layers(w, 1)
    # selected pairs against the closed-form n log n total for power-of-two lengths
    m = int(np.log2(n // 64))
    assert int(route.total_pairs.item()) == n * 64 * m - 64 * 64 * m + n * 65 // 2
    rows = sample_rows(w, per_seq=200)
    print(name, "bf1", check(w, inputs, outs, lses, rows))
    inputs, outs, lses, _ = gpu_layers(w, 1, dense=True)
    rows_d = sample_rows(w, per_seq=60)
    print(name, "dense", check(w, inputs, outs, lses, rows_d, dense=True))


def test_dense_mode_32k_sampled():
    w = I.WORKLOADS["qwen_32k"]
    inputs, outs, lses, _ = gpu_layers(w, 1, dense=True)
    rows = sample_rows(w, per_seq=40)
    print("32k dense", check(w, inputs, outs, lses, rows, dense=True))


def test_ragged_batch_single_varlen_launch():
    w = I.WORKLOADS["ragged"]
    inputs, outs, lses, route = gpu_layers(w, 1)
    assert int(route.num_qblocks.item()) == 47 + 128 + 193 + 256
    assert int(route.total_pairs.item()) == 1_155_061 + 3_907_584 + 6_430_389 + 8_888_320
    rows = sample_rows(w, per_seq=150)
    # the partial last blocks (57 rows each) of sequences 0 and 2, row by row
    cu = w.cu_seqlens()
    tails = np.concatenate([np.arange(cu[1] - 57, cu[1]), np.arange(cu[3] - 57, cu[3])])
    rows = np.unique(np.concatenate([rows, tails]))
    print("ragged", check(w, inputs, outs, lses, rows))
    # one varlen launch equals four separate launches, bit for bit
    o, lse = outs[0], lses[0]
    q, k, v = inputs[0]
    for s, n in enumerate(w.seqlens):
        sl = slice(cu[s], cu[s + 1])
        w1 = I.custom([n], hq=w.hq, hkv=w.hkv, d=w.d, seed=0)
        dev = torch.device("cuda:0")
        cu1 = bf1.cu_seqlens_tensor([n], dev)
        r1 = bf1.plan_route(cu1, n)
        o1, l1 = bf1.attn_fwd(q[sl].contiguous().to(dev), k[sl].contiguous().to(dev), v[sl].contiguous().to(dev),
                              cu1, n, r1)
        torch.cuda.synchronize()
        assert np.array_equal(o[sl], o1.float().cpu().numpy()) and np.array_equal(lse[:, sl], l1.cpu().numpy())
