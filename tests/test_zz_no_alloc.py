"""bf1_attn_fwd_noalloc: the entry point for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is unavailable -- after a server has fixed
its memory budget, in a real-time loop, under an allocator that must not be re-entered.  For
them the library keeps the route arrays and the kernel's hand-out counters in a fixed array of
its own.  These tests call that entry point through the C ABI twice in a row (the second call
finds the first call's leftovers in the shared array, once from a larger batch) and compare with
the CPU oracle at the stated tolerances and, bit for bit, with what bf1_plan_route + bf1_attn_fwd
produce for the same inputs (same kernel, same lists: any difference would be a stale or
misplaced scratch entry).  The file sorts last on purpose, so that a run which
stops at the first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import bf1_inputs as I
import paper_2608_20427_b200 as bf1

from oracle import bf1_oracle as O

from gpu_util import assert_parity, oracle_cfg


def test_requests_beyond_the_built_in_scratch_are_refused_on_the_host():
    lib = bf1.load()
    fake = ctypes.c_void_p(0x1000)
    cfg = bf1.RouteCfg()
    # 4097 query blocks: one more than the scratch holds
    n = 4097 * 64
    rc = lib.bf1_attn_fwd_noalloc(fake, fake, fake, fake, 1, n, n, 16, 8, 128, 0.0, ctypes.byref(cfg), fake, fake,
                                  None, None)
    assert rc == -3 and b"4096" in lib.bf1_last_error()
    # lists longer than 32 entries
    wide = bf1.RouteCfg(local_blocks=40)
    rc = lib.bf1_attn_fwd_noalloc(fake, fake, fake, fake, 1, 64 * 100, 64 * 100, 16, 8, 128, 0.0, ctypes.byref(wide),
                                  fake, fake, None, None)
    assert rc == -3 and b"32" in lib.bf1_last_error()
    # geometry and pointer errors come before the capacity check and before anything is launched
    rc = lib.bf1_attn_fwd_noalloc(fake, fake, fake, fake, 1, n, n, 16, 2, 128, 0.0, ctypes.byref(cfg), fake, fake,
                                  None, None)
    assert rc == -2 and b"group" in lib.bf1_last_error()
    rc = lib.bf1_attn_fwd_noalloc(None, fake, fake, fake, 1, 64, 64, 16, 8, 128, 0.0, ctypes.byref(cfg), fake, fake,
                                  None, None)
    assert rc == -1


def test_the_documented_limit_itself_is_accepted():
    """The block count the entry point checks is bf1_route_capacity's bound.  One sequence of 262,144
    tokens is exactly 4096 blocks and must not be counted as 4097; a batch of B sequences may end in B
    partial blocks, so its bound is B + floor((T - B) / 64)."""
    assert bf1.route_capacity(1, 4096 * 64, 4096 * 64)[0] == 4096
    assert bf1.route_capacity(1, 4096 * 64 + 1, 4096 * 64 + 1)[0] == 4097
    assert bf1.route_capacity(1, 4096 * 64 - 63, 4096 * 64)[0] == 4096
    assert bf1.route_capacity(4, 64 * (4096 - 4) + 4, 262144)[0] == 4096
    assert bf1.route_capacity(4, 64 * (4096 - 4) + 5, 262144)[0] == 4096      # 4 partial blocks + 4092 full, 1 token spare
    assert bf1.route_capacity(4, 64 * (4096 - 3) + 4, 262144)[0] == 4097
    assert bf1.route_capacity(3, 2, 2)[0] == 2                                # more sequences than tokens
    # brute force on small cases: the bound is attained and never exceeded
    import functools

    @functools.lru_cache(maxsize=None)
    def most_blocks(batch, total):
        if batch == 1:
            return (total + 63) // 64
        return max((x + 63) // 64 + most_blocks(batch - 1, total - x) for x in range(total + 1))

    for batch in (1, 2, 3):
        for total in range(0, 200):
            assert bf1.route_capacity(batch, total, max(total, 1))[0] == max(most_blocks(batch, total), 1), (batch, total)


@pytest.mark.gpu
def test_two_calls_in_a_row_match_the_oracle_and_the_allocating_entry_points_bitwise():
    dev = torch.device("cuda:0")
    cases = [I.custom([3001, 0, 257, 4096], hq=4, hkv=2, d=128, seed=2101),   # ragged batch: 117 query blocks
             I.custom([1000], hq=2, hkv=1, d=64, seed=2100)]                  # then a small one: 16 blocks, the
                                                                              # rest of the array holds leftovers
    # everything either path needs is allocated here, before the window in which nothing may be allocated
    prepared = []
    for w in cases:
        q, k, v = I.draw_qkv(w)
        qd, kd, vd = (t.to(dev) for t in (q, k, v))
        cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
        T = w.total_tokens
        route = bf1.plan_route(cu, w.max_seqlen)
        o_alloc, lse_alloc = bf1.attn_fwd(qd, kd, vd, cu, w.max_seqlen, route)
        torch.cuda.synchronize()
        route.check_status()
        outs = [torch.full((T, w.hq, w.d), float("nan"), dtype=torch.bfloat16, device=dev) for _ in range(2)]
        lses = [torch.full((w.hq, T), float("nan"), dtype=torch.float32, device=dev) for _ in range(2)]
        prepared.append((w, q, k, v, qd, kd, vd, cu, o_alloc, lse_alloc, outs, lses))
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    # one call up front: the library looks up its array and CUDA loads the kernels on first use
    w, q, k, v, qd, kd, vd, cu, _, _, outs, lses = prepared[1]
    bf1.attn_fwd_noalloc(qd, kd, vd, cu, w.max_seqlen, outs[0], lses[0], status=status)
    torch.cuda.synchronize()
    outs[0].fill_(float("nan"))
    lses[0].fill_(float("nan"))
    torch.cuda.synchronize()
    # ---- the window: two calls per case, back to back; neither torch's allocator nor the driver's
    #      free-memory figure (which also sees a cudaMalloc made inside the library) may move
    free_before = torch.cuda.mem_get_info(dev)[0]
    torch_before = torch.cuda.memory_allocated(dev)
    for w, q, k, v, qd, kd, vd, cu, _, _, outs, lses in prepared:
        for rep in range(2):
            bf1.attn_fwd_noalloc(qd, kd, vd, cu, w.max_seqlen, outs[rep], lses[rep], status=status)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated(dev) == torch_before
    assert torch.cuda.mem_get_info(dev)[0] == free_before
    assert int(status.item()) == 0
    for w, q, k, v, qd, kd, vd, cu, o_alloc, lse_alloc, outs, lses in prepared:
        o_ref, lse_ref = O.attn_route(oracle_cfg(w), q, k, v, w.cu_seqlens())
        for rep in range(2):
            assert_parity(outs[rep].float().cpu().numpy(), lses[rep].cpu().numpy(), o_ref, lse_ref)
            assert torch.equal(outs[rep], o_alloc) and torch.equal(lses[rep], lse_alloc), (w.seqlens, rep)
    # without a caller-owned status word the device status stays inside the library
    w, q, k, v, qd, kd, vd, cu, o_alloc, lse_alloc, outs, lses = prepared[0]
    outs[0].fill_(float("nan"))
    bf1.attn_fwd_noalloc(qd, kd, vd, cu, w.max_seqlen, outs[0], lses[0])
    torch.cuda.synchronize()
    assert torch.equal(outs[0], o_alloc) and torch.equal(lses[0], lse_alloc)
