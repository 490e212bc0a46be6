"""Gradients of the routed attention on the GPU vs the fp64 CPU oracle (Section 4.2's gradient gate).  The
kernels round P and dS to bf16 before their MMAs and their outputs to bf16, so the comparison is by relative RMS
and by the largest error relative to the gradient's scale.  Nothing is added with atomics: the three gradients
must come out bit-identical on every run."""
import numpy as np
import pytest
import torch

import bf1_inputs as I
import paper_2608_20427_b200 as bf1
from oracle import bf1_oracle as O

from gpu_util import oracle_cfg, lib_cfg

pytestmark = pytest.mark.gpu
REL_RMS = 1e-2          # P, dS and the outputs are bf16 (2^-9 relative each); observed 2e-3 .. 5e-3
REL_MAX = 2e-2          # of the gradient's largest magnitude; observed <= 6e-3
ZERO_ABS = 1e-4         # where the exact gradient is zero: fp32 rounding of O(10) dot products, times P <= 1


def run_case(w, seed):
    dev = torch.device("cuda:0")
    q, k, v = I.draw_qkv(w)
    g = torch.Generator().manual_seed(seed)
    d_o = torch.randn(q.shape, generator=g).to(torch.bfloat16)
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
    route = bf1.plan_route(cu, w.max_seqlen, lib_cfg(w))
    qd, kd, vd, gd = q.to(dev), k.to(dev), v.to(dev), d_o.to(dev)
    o, lse = bf1.attn_fwd(qd, kd, vd, cu, w.max_seqlen, route)
    dq, dk, dv = bf1.attn_bwd(qd, kd, vd, o, lse, gd, cu, w.max_seqlen, route)
    torch.cuda.synchronize()
    route.check_status()
    rq, rk, rv = O.attn_route_bwd(oracle_cfg(w), q, k, v, d_o.float().numpy().astype(np.float64), w.cu_seqlens())
    out = {}
    for name, got, ref in (("dq", dq, rq), ("dk", dk, rk), ("dv", dv, rv)):
        got = got.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all(), name
        diff = got - ref
        scale = float(np.abs(ref).max())
        if scale < 1e-9:
            # a gradient that is zero by definition (a token whose only key is itself has dq = dk = 0):
            # the kernel's D = <dO, O> and dP = <dO, V> differ by fp32 rounding only, so what is left
            # must be tiny in absolute terms -- no relative floor to hide behind
            assert float(np.abs(got).max()) <= ZERO_ABS, (name, float(np.abs(got).max()))
            out[name] = (0.0, 0.0)
            continue
        rms_ref = float(np.sqrt((ref ** 2).mean()))
        out[name] = (float(np.sqrt((diff ** 2).mean())) / rms_ref, float(np.abs(diff).max()) / scale)
    return out


@pytest.mark.parametrize("lens", [[64], [1], [65], [257], [1000], [130, 0, 257, 64, 1, 700]],
                         ids=lambda x: "-".join(map(str, x)))
def test_gradients_match_the_oracle(lens):
    w = I.custom(lens, hq=4, hkv=2, d=128, seed=6000 + sum(lens))
    res = run_case(w, seed=1)
    print(lens, res)
    for name, (rms, mx) in res.items():
        assert rms <= REL_RMS and mx <= REL_MAX, (name, rms, mx)


def test_gradients_4k_qwen_geometry():
    w = I.custom([4096], hq=16, hkv=8, d=128, seed=6100, sink_scale=4.0)
    res = run_case(w, seed=2)
    print("4k", res)
    for name, (rms, mx) in res.items():
        assert rms <= REL_RMS and mx <= REL_MAX, (name, rms, mx)


@pytest.mark.parametrize("n", [8192, 32768])
def test_gradients_at_the_benchmarked_lengths(n):
    """The sizes bench.py's `backward` block times: several waves of units, lists of 9 to 11 entries,
    up to eleven query blocks adding into one KV block.  All of dQ, dK, dV against the fp64 oracle."""
    w = I.custom([n], hq=16, hkv=8, d=128, seed=6200 + n)
    res = run_case(w, seed=3)
    print(n, res)
    for name, (rms, mx) in res.items():
        assert rms <= REL_RMS and mx <= REL_MAX, (name, rms, mx)


@pytest.mark.parametrize("hq,hkv,d", [(4, 2, 64), (8, 2, 128), (8, 2, 64), (3, 3, 128), (2, 2, 64)],
                         ids=["G2-d64", "G4-d128", "G4-d64", "G1-d128", "G1-d64"])
def test_gradients_in_every_geometry_the_forward_takes(hq, hkv, d):
    """Section 4.2's gradient gate per geometry: head dimension 64, four query heads per KV head (two CTAs per unit
    whose dK / dV contributions add up), one query head per KV head (half of the tile idle)."""
    for lens in ([1, 65, 257, 1000], [2500]):
        w = I.custom(lens, hq=hq, hkv=hkv, d=d, seed=6300 + hq + d + len(lens))
        res = run_case(w, seed=4)
        print(hq, hkv, d, lens, res)
        for name, (rms, mx) in res.items():
            assert rms <= REL_RMS and mx <= REL_MAX, (name, rms, mx)


@pytest.mark.parametrize("route", [dict(local_blocks=9, global_first=0, dyadic=0),      # sliding window: ten readers per block
                                   dict(local_blocks=40, global_first=1, dyadic=1),     # 41+ readers per block: cut into runs
                                   dict(local_blocks=0, global_first=0, dyadic=1)],     # dyadic predecessors only
                         ids=["sliding", "wide", "dyadic-only"])
def test_gradients_over_other_routes(route):
    """dK / dV walk the INVERSE of whatever lists the route holds; these routes give it other shapes than BF1's."""
    w = I.custom([4096, 700], hq=4, hkv=2, d=128, seed=6400, **route)
    res = run_case(w, seed=5)
    print(route, res)
    for name, (rms, mx) in res.items():
        assert rms <= REL_RMS and mx <= REL_MAX, (name, rms, mx)


def test_gradients_of_many_short_sequences():
    """Hundreds of sequences of one to three blocks: more units than the persistent kernels have CTAs, nearly all of
    one or two list entries, so every ring, buffer pair and barrier phase changes hands at every step; units of
    sequences with a single token have nothing but the self block."""
    rng = np.random.default_rng(77)
    lens = [int(x) for x in rng.integers(1, 190, size=700)]
    lens[5] = 0
    lens[100:108] = [1, 64, 65, 128, 129, 1, 63, 2]
    w = I.custom(lens, hq=4, hkv=2, d=64, seed=6600)
    res = run_case(w, seed=7)
    print(len(lens), sum(lens), res)
    for name, (rms, mx) in res.items():
        assert rms <= REL_RMS and mx <= REL_MAX, (name, rms, mx)


def test_gradients_over_a_dense_route():
    """Every predecessor selected (lists of up to 32 entries, every block with many readers): long units in the dQ
    kernel, every KV block of the first half cut into runs in the dK/dV kernel."""
    w = I.custom([2048], hq=4, hkv=2, d=128, seed=6700, local_blocks=64, global_first=1, dyadic=1)
    res = run_case(w, seed=8)
    print(res)
    for name, (rms, mx) in res.items():
        assert rms <= REL_RMS and mx <= REL_MAX, (name, rms, mx)


def test_backward_over_a_damaged_route_is_the_backward_of_the_repaired_route():
    """Entries outside [0, j], a list that does not end in its query block, counts past the pitch: every kernel of the
    library reads a list the same repaired way (the forward flags it), so the gradients over the damaged route are,
    bit for bit, those over the route with the repairs written in -- and nothing faults."""
    dev = torch.device("cuda:0")
    w = I.custom([1500, 300], hq=4, hkv=2, d=128, seed=6800)
    q, k, v = (t.to(dev) for t in I.draw_qkv(w))
    d_o = torch.randn(q.shape, generator=torch.Generator().manual_seed(9)).to(torch.bfloat16).to(dev)
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)

    def grads(damage):
        route = bf1.plan_route(cu, w.max_seqlen)
        deg = route.max_degree
        cnt = route.kv_count.cpu()
        blk = route.qb_block.cpu()
        idx = route.kv_idx.cpu().clone()
        kc = cnt.clone()
        g1, g2, g3 = 7, 12, 20            # slots of the first sequence (24 blocks)
        if damage:
            idx[g1, 0] = 1000             # out of range            -> read as block 0
            idx[g2, 1] = -5               # negative                -> read as block 0
            idx[g3, int(cnt[g3]) - 1] = 3 # last entry not the self block -> read as the self block
            kc[g2] = deg + 50             # count past the pitch    -> cut to the pitch
        else:
            idx[g1, 0] = 0
            idx[g2, 1] = 0
            idx[g3, int(cnt[g3]) - 1] = int(blk[g3])
            # kc[g2] cut to the pitch: the entries past the old count are the -1 padding, read as block 0, and the
            # last one as the self block
            kc[g2] = deg
            idx[g2, int(cnt[g2]) - 1] = 0
            idx[g2, int(cnt[g2]):deg - 1] = 0
            idx[g2, deg - 1] = int(blk[g2])
        route.kv_idx.copy_(idx.to(dev))
        route.kv_count.copy_(kc.to(dev))
        o, lse = bf1.attn_fwd(q, k, v, cu, w.max_seqlen, route)
        out = bf1.attn_bwd(q, k, v, o, lse, d_o, cu, w.max_seqlen, route)
        torch.cuda.synchronize()
        return out, int(route.status.item())

    bad, status_bad = grads(True)
    good, status_good = grads(False)
    assert status_bad & 8 and not status_good & 8
    for x, y in zip(bad, good):
        assert torch.isfinite(x.float()).all()
        assert torch.equal(x, y)


def test_backward_is_bitwise_reproducible():
    """No floating-point atomics: two runs give the same bits, whatever the workspace held before (block 0 of the
    long sequence has 64 readers and goes through the partial-sum path)."""
    dev = torch.device("cuda:0")
    w = I.custom([4096, 1000, 65], hq=8, hkv=2, d=128, seed=6500)
    q, k, v = (t.to(dev) for t in I.draw_qkv(w))
    d_o = torch.randn(q.shape, generator=torch.Generator().manual_seed(6)).to(torch.bfloat16).to(dev)
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
    route = bf1.plan_route(cu, w.max_seqlen)
    o, lse = bf1.attn_fwd(q, k, v, cu, w.max_seqlen, route)
    ws = bf1.bwd_workspace(route, w.total_tokens, w.hq, w.hkv, w.d, dev)
    runs = []
    for fill in (0x00, 0xFF, 0x7F):          # 0xFF bytes are NaNs as fp32, 0x7F.. huge ints as counters
        ws.fill_(fill)
        runs.append(bf1.attn_bwd(q, k, v, o, lse, d_o, cu, w.max_seqlen, route, workspace=ws))
        torch.cuda.synchronize()
        route.check_status()
    for other in runs[1:]:
        for x, y in zip(runs[0], other):
            assert torch.equal(x, y)
    assert all(torch.isfinite(t.float()).all() for t in runs[0])


def test_backward_rejects_what_it_does_not_support():
    dev = torch.device("cuda:0")
    w = I.custom([128], hq=2, hkv=1, d=64, seed=1)
    q, k, v = (t.to(dev) for t in I.draw_qkv(w))
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
    route = bf1.plan_route(cu, 128)
    o, lse = bf1.attn_fwd(q, k, v, cu, 128, route)
    lib = bf1.load()
    rc = lib.bf1_attn_bwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), q.data_ptr(),
                          cu.data_ptr(), 1, 128, 128, 6, 1, 64, 0.0, route.c, q.data_ptr(), q.data_ptr(), q.data_ptr(),
                          q.data_ptr(), None)
    assert rc == -2 and b"group" in lib.bf1_last_error()      # G = 6
    rc = lib.bf1_attn_bwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), q.data_ptr(),
                          cu.data_ptr(), 1, 128, 128, 2, 1, 96, 0.0, route.c, q.data_ptr(), q.data_ptr(), q.data_ptr(),
                          q.data_ptr(), None)
    assert rc == -2 and b"dimension" in lib.bf1_last_error()  # d = 96
