"""Cached one-token decode over selected pages (Section 3.2, Section 5.4) vs the CPU oracle.

The oracle for a decode step is the last row of the routed attention over the same (logical) keys
and values: the newest token reads P(block of n-1), the self block up to itself.  The gates are the
paper's: agreement with that reference, tail handling, page-permutation invariance, zero decoy-page
leakage, and one plan serving a whole 64-token route epoch."""
import numpy as np
import pytest
import torch

import bf1_inputs as I
import paper_2608_20427_b200 as bf1
from oracle import bf1_oracle as O

from gpu_util import LSE_ABS, O_MAX_ABS, O_REL_RMS

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def paged_cache(w, k, v, seed, decoys=7, decoy_scale=50.0):
    """Scatter the logical K/V of a packed batch into randomly permuted physical pages, with decoy
    pages (large finite garbage) in between.  Returns k_pages, v_pages, page_table (CPU tensors)."""
    g = torch.Generator().manual_seed(seed)
    blocks = [(n + 63) // 64 for n in w.seqlens]
    total = sum(blocks) + decoys
    perm = torch.randperm(total, generator=g)
    k_pages = (torch.randn((total, 64, w.hkv, w.d), generator=g) * decoy_scale).to(torch.bfloat16)
    v_pages = (torch.randn((total, 64, w.hkv, w.d), generator=g) * decoy_scale).to(torch.bfloat16)
    table = torch.full((len(blocks), max(max(blocks), 1)), -1, dtype=torch.int32)
    cu = w.cu_seqlens()
    nxt = 0
    for s, nb in enumerate(blocks):
        for b in range(nb):
            pg = int(perm[nxt]); nxt += 1
            table[s, b] = pg
            lo, hi = cu[s] + 64 * b, min(cu[s] + 64 * b + 64, cu[s + 1])
            k_pages[pg, :hi - lo] = k[lo:hi]
            v_pages[pg, :hi - lo] = v[lo:hi]
    return k_pages, v_pages, table


def run_decode(w, q, k_pages, v_pages, table, seqlens=None, plan=None):
    dev = torch.device(DEV)
    sl = torch.tensor(list(w.seqlens if seqlens is None else seqlens), dtype=torch.int32, device=dev)
    cu = w.cu_seqlens()
    last = [cu[s] + (n - 1) for s, n in enumerate(sl.tolist())]
    qd = torch.stack([q[i] if n > 0 else torch.zeros_like(q[0]) for i, n in zip(last, sl.tolist())]).to(dev)
    tb = table.to(dev)
    if plan is None:
        plan = bf1.plan_decode(sl, tb)
    ws = bf1.decode_workspace(len(w.seqlens), w.hq, w.hkv, plan.max_degree, w.d, dev)
    out = torch.full((len(w.seqlens), w.hq, w.d), float("nan"), dtype=torch.bfloat16, device=dev)
    lse = torch.full((w.hq, len(w.seqlens)), float("nan"), dtype=torch.float32, device=dev)
    for _ in range(2):   # twice: the second call finds the ticket words the first one left
        bf1.decode_fwd(qd, k_pages.to(dev), v_pages.to(dev), sl, plan, ws, out=out, lse=lse)
    torch.cuda.synchronize()
    pairs = (w.hq // w.hkv + 1) // 2
    assert int(ws.view(torch.int32)[-len(w.seqlens) * w.hkv * pairs:].abs().sum().item()) == 0
    return out.float().cpu().numpy(), lse.cpu().numpy(), plan, last


def check(w, q, k, v, out, lse, last):
    rows = [r for r, n in zip(last, w.seqlens) if n > 0]
    o_ref, lse_ref = O.attn_route(O.cfg(), q, k, v, w.cu_seqlens(), rows=rows)
    live = [s for s, n in enumerate(w.seqlens) if n > 0]
    diff = out[live].astype(np.float64) - o_ref[rows]
    assert not np.isnan(out[live]).any() and not np.isnan(lse[:, live]).any()
    assert np.abs(diff).max() <= O_MAX_ABS
    assert np.sqrt((diff ** 2).mean() / (o_ref[rows].astype(np.float64) ** 2).mean()) <= O_REL_RMS
    assert np.abs(lse[:, live] - lse_ref[:, rows]).max() <= LSE_ABS


@pytest.mark.parametrize("d", [64, 128])
def test_decode_matches_oracle_with_tails_and_empty_sequences(d):
    lens = [1, 64, 65, 257, 1000, 0, 4097, 12345]
    w = I.custom(lens, hq=4, hkv=2, d=d, seed=3000 + d)
    q, k, v = I.draw_qkv(w)
    k_pages, v_pages, table = paged_cache(w, k, v, seed=1)
    out, lse, plan, last = run_decode(w, q, k_pages, v_pages, table)
    assert int(plan.status.item()) == 0
    check(w, q, k, v, out, lse, last)
    # the plan: physical pages of Eq. 1's list for the newest token's block, self page last
    cnt, pages = plan.count.cpu().numpy(), plan.page.cpu().numpy()
    for s, n in enumerate(lens):
        if n == 0:
            assert cnt[s] == 0 and np.isnan(out[s]).all()
            continue
        j = (n - 1) // 64
        idx, c, _, _ = O.route(O.cfg(), n, plan.max_degree)
        want = [int(table[s, b]) for b in idx[j, :c[j]]]
        assert cnt[s] == c[j] and list(pages[s, :cnt[s]]) == want and (pages[s, cnt[s]:] == -1).all()


def test_long_context_decode_32k_and_64k():
    w = I.custom([32768, 65536], hq=16, hkv=8, d=128, seed=3100)
    q, k, v = I.draw_qkv(w)
    k_pages, v_pages, table = paged_cache(w, k, v, seed=2)
    out, lse, plan, last = run_decode(w, q, k_pages, v_pages, table)
    assert plan.count.tolist() == [11, 12]      # 3 + floor(log2 511), 3 + floor(log2 1023)
    check(w, q, k, v, out, lse, last)


@pytest.mark.parametrize("d", [64, 128])
def test_large_batch_takes_the_one_cta_per_list_path(d):
    """batch x KV heads >= number of SMs: one CTA walks a whole page list with an online softmax."""
    rng = np.random.default_rng(7)
    lens = [int(x) for x in rng.integers(1, 3000, size=40)] + [1, 64, 65, 0, 4097]
    w = I.custom(lens, hq=8, hkv=4, d=d, seed=3500 + d)    # 45 x 4 = 180 pairs
    q, k, v = I.draw_qkv(w)
    k_pages, v_pages, table = paged_cache(w, k, v, seed=5)
    out, lse, plan, last = run_decode(w, q, k_pages, v_pages, table)
    assert int(plan.status.item()) == 0
    check(w, q, k, v, out, lse, last)
    # NaN behind the newest token and in unselected pages must not leak on this path either
    used = set(int(x) for x in table.flatten().tolist() if x >= 0)
    for pg in range(k_pages.shape[0]):
        if pg not in used:
            k_pages[pg] = float("nan")
            v_pages[pg] = float("nan")
    for s_, n_ in enumerate(w.seqlens):
        if n_ % 64:
            pg = int(table[s_, (n_ - 1) // 64])
            k_pages[pg, n_ % 64:] = float("nan")
            v_pages[pg, n_ % 64:] = float("nan")
    out1, lse1, _, _ = run_decode(w, q, k_pages, v_pages, table)
    live = [i for i, n_ in enumerate(lens) if n_ > 0]
    assert np.array_equal(out[live], out1[live]) and np.array_equal(lse[:, live], lse1[:, live])


def test_page_permutation_invariance_and_zero_decoy_leakage():
    w = I.custom([700, 3001], hq=4, hkv=2, d=128, seed=3200)
    q, k, v = I.draw_qkv(w)
    ref = None
    for seed, scale in ((10, 50.0), (11, 50.0), (10, 1000.0)):   # another permutation; other decoy contents
        k_pages, v_pages, table = paged_cache(w, k, v, seed=seed, decoy_scale=scale)
        out, lse, _, _ = run_decode(w, q, k_pages, v_pages, table)
        if ref is None:
            ref = (out, lse)
        assert np.array_equal(out, ref[0]) and np.array_equal(lse, ref[1])


def test_unwritten_page_tails_may_hold_anything():
    """The part of the newest page behind the newest token is unwritten cache memory: NaN there
    (and in pages the route does not select) must not reach the output."""
    w = I.custom([1000, 65], hq=4, hkv=2, d=128, seed=3400)
    q, k, v = I.draw_qkv(w)
    k_pages, v_pages, table = paged_cache(w, k, v, seed=4)
    out0, lse0, _, _ = run_decode(w, q, k_pages, v_pages, table)
    used = set(int(x) for x in table.flatten().tolist() if x >= 0)
    for pg in range(k_pages.shape[0]):
        if pg not in used:
            k_pages[pg] = float("nan")
            v_pages[pg] = float("nan")
    for s, n in enumerate(w.seqlens):
        tail = n % 64
        if tail:
            pg = int(table[s, (n - 1) // 64])
            k_pages[pg, tail:] = float("nan")
            v_pages[pg, tail:] = float("nan")
    out1, lse1, _, _ = run_decode(w, q, k_pages, v_pages, table)
    assert np.array_equal(out0, out1) and np.array_equal(lse0, lse1)


def test_one_plan_serves_a_route_epoch_and_refuses_the_next():
    n0 = 64 * 9 + 1                                       # first token of block 9
    w = I.custom([n0 + 63], hq=4, hkv=2, d=128, seed=3300)
    q, k, v = I.draw_qkv(w)
    k_pages, v_pages, table = paged_cache(w, k, v, seed=3)
    dev = torch.device(DEV)
    plan = bf1.plan_decode(torch.tensor([n0], dtype=torch.int32, device=dev), table.to(dev))
    for n in (n0, n0 + 1, n0 + 31, n0 + 63):              # same plan, growing tail
        wn = I.custom([n], hq=4, hkv=2, d=128, seed=0)
        out, lse, _, last = run_decode(wn, q[:n], k_pages, v_pages, table, plan=plan)
        assert int(plan.status.item()) == 0
        check(wn, q[:n], k[:n], v[:n], out, lse, last)
    # one token further the newest token lives in block 10: the stale plan is flagged, nothing is read
    dev_sl = torch.tensor([n0 + 64], dtype=torch.int32, device=dev)
    ws = bf1.decode_workspace(1, 4, 2, plan.max_degree, 128, dev)
    bf1.decode_fwd(q[:1].to(dev), k_pages.to(dev), v_pages.to(dev), dev_sl, plan, ws)
    torch.cuda.synchronize()
    assert int(plan.status.item()) & 8


def test_decode_plan_flags_a_sequence_longer_than_its_page_table():
    dev = torch.device(DEV)
    table = torch.zeros((1, 4), dtype=torch.int32, device=dev)
    plan = bf1.plan_decode(torch.tensor([4 * 64 + 1], dtype=torch.int32, device=dev), table)
    torch.cuda.synchronize()
    assert int(plan.status.item()) & 1 and int(plan.count.item()) == 0


@pytest.mark.parametrize("hq,hkv", [(8, 2), (3, 3)], ids=["G4", "G1"])
@pytest.mark.parametrize("batch_kind", ["few", "many"])
def test_decode_with_four_and_with_one_query_head_per_kv_head(hq, hkv, batch_kind):
    """G = 4 runs two CTAs (pairs of query heads) per KV head, G = 1 half a pair; both forms of the kernel
    are exercised: lists cut into runs with a combine (few sequences) and one CTA per list (many)."""
    lens = [1, 64, 65, 257, 1000, 0, 4097] if batch_kind == "few" else [1 + (37 * i) % 700 for i in range(90)]
    w = I.custom(lens, hq=hq, hkv=hkv, d=128, seed=7100 + hq + len(lens))
    q, k, v = I.draw_qkv(w)
    k_pages, v_pages, table = paged_cache(w, k, v, seed=7200 + hq)
    out, lse, plan, last = run_decode(w, q, k_pages, v_pages, table)
    assert int(plan.status.item()) == 0
    check(w, q, k, v, out, lse, last)
