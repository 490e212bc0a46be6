"""Helpers shared by the GPU parity tests: run the CUDA path on a workload, run the oracle,
compare with the tolerances the benchmark spec states (max-abs 2e-2, relative RMS 1e-2 on O; 1e-3 on LSE)."""
import numpy as np
import torch

import bf1_inputs as I
import paper_2608_20427_b200 as bf1
from oracle import bf1_oracle as O

O_MAX_ABS = 2e-2
O_REL_RMS = 1e-2
LSE_ABS = 1e-3


def oracle_cfg(w):
    return O.cfg(w.block, w.local_blocks, w.global_first, w.dyadic)


def lib_cfg(w):
    return bf1.RouteCfg(w.block, w.local_blocks, w.global_first, w.dyadic)


def poison(shape, dtype, device):
    """NaN-filled output buffer: a row the kernel forgets to write cannot pass for a result."""
    return torch.full(shape, float("nan"), dtype=dtype, device=device)


def run_gpu(w, q, k, v, dense=False, scale=None, guard=0):
    """Run the CUDA path.  `guard` extra token rows after the batch are poisoned and must stay so."""
    dev = torch.device("cuda:0")
    T = w.total_tokens
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
    out = poison((T + guard, w.hq, w.d), torch.bfloat16, dev)
    lse = poison((w.hq, T), torch.float32, dev)
    if dense:
        work = torch.zeros(4, dtype=torch.int32, device=dev)
        bf1.dense_causal_fwd(qd, kd, vd, cu, w.max_seqlen, scale=scale, out=out[:T], lse=lse, work=work)
        torch.cuda.synchronize()
        assert work.tolist() == [0, 0, 0, 0]
        route = None
    else:
        route = bf1.plan_route(cu, w.max_seqlen, lib_cfg(w))
        bf1.attn_fwd(qd, kd, vd, cu, w.max_seqlen, route, scale=scale, out=out[:T], lse=lse)
        torch.cuda.synchronize()
        route.check_status()
        assert route.sched.tolist() == [0, 0]   # hand-out counters are back at zero
    if guard:
        assert torch.isnan(out[T:].float()).all(), "kernel wrote past the last token row"
    return out[:T].float().cpu().numpy(), lse.cpu().numpy(), route


def errors(o_gpu, lse_gpu, o_ref, lse_ref, rows=None):
    if rows is not None:
        o_gpu, o_ref = o_gpu[rows], o_ref[rows]
        lse_gpu, lse_ref = lse_gpu[:, rows], lse_ref[:, rows]
    diff = o_gpu.astype(np.float64) - o_ref.astype(np.float64)
    return {
        "o_max_abs": float(np.abs(diff).max()) if diff.size else 0.0,
        "o_rel_rms": float(np.sqrt((diff ** 2).mean() / max((o_ref.astype(np.float64) ** 2).mean(), 1e-30))) if diff.size else 0.0,
        "lse_max_abs": float(np.abs(lse_gpu.astype(np.float64) - lse_ref).max()) if lse_ref.size else 0.0,
        "o_absmax_ref": float(np.abs(o_ref).max()) if o_ref.size else 0.0,
    }


def assert_parity(o_gpu, lse_gpu, o_ref, lse_ref, rows=None):
    assert not np.isnan(o_gpu if rows is None else o_gpu[rows]).any(), "unwritten or NaN output rows"
    assert not np.isnan(lse_gpu if rows is None else lse_gpu[:, rows]).any(), "unwritten or NaN LSE"
    e = errors(o_gpu, lse_gpu, o_ref, lse_ref, rows)
    assert e["o_max_abs"] <= O_MAX_ABS, e
    assert e["o_rel_rms"] <= O_REL_RMS, e
    assert e["lse_max_abs"] <= LSE_ABS, e
    return e


def host_route(lists_per_seq, seqlens, max_degree=None, block=64):
    """Route arrays for `bf1.Route.from_host`, written by hand on the host from explicit lists
    (one list of ascending KV block indices per query block, self block last): slots numbered
    sequence by sequence, pair counts by Proposition 1's accounting, hand-out order by
    descending list length.  Returns (arrays dict, total_pairs)."""
    qb_seq, qb_block, counts, pairs, rows_idx = [], [], [], [], []
    for s, (lists, n) in enumerate(zip(lists_per_seq, seqlens)):
        assert len(lists) == (n + block - 1) // block
        for j, lst in enumerate(lists):
            assert lst == sorted(set(lst)) and lst[-1] == j and lst[0] >= 0
            rows = min(block, n - j * block)
            qb_seq.append(s)
            qb_block.append(j)
            counts.append(len(lst))
            pairs.append(rows * block * (len(lst) - 1) + rows * (rows + 1) // 2)
            rows_idx.append(lst)
    deg = max_degree or max(counts)
    kv_idx = np.full((len(counts), deg), -1, dtype=np.int32)
    for g, lst in enumerate(rows_idx):
        kv_idx[g, :len(lst)] = lst
    order = sorted(range(len(counts)), key=lambda g: (-counts[g], g))
    arrays = dict(qb_seq=qb_seq, qb_block=qb_block, kv_count=counts, kv_idx=kv_idx, pair_count=pairs, order=order)
    return arrays, int(sum(pairs))


def mask_from_lists(lists, n, block=64):
    """n x n boolean token mask of one sequence: listed blocks in full, the self block causally."""
    m = np.zeros((n, n), dtype=bool)
    for j, lst in enumerate(lists):
        r0, r1 = j * block, min((j + 1) * block, n)
        for p in lst:
            c0, c1 = p * block, min((p + 1) * block, n)
            m[r0:r1, c0:c1] = True
    return m & np.tril(np.ones((n, n), dtype=bool))
