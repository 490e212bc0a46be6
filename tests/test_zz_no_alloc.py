"""bf1_attn_fwd_noalloc: the entry point for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is unavailable -- after a server has fixed
its memory budget, in a real-time loop, under an allocator that must not be re-entered.  For
them the library keeps the route arrays and the kernel's hand-out counters in a fixed array of
its own.  These tests call that entry point through the C ABI twice in a row (the second call
finds the first call's leftovers in the shared array) and compare with what bf1_plan_route +
bf1_attn_fwd produce for the same inputs.  The file sorts last on purpose, so that a run which
stops at the first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import bf1_inputs as I
import paper_2608_20427_b200 as bf1

from gpu_util import LSE_ABS, O_MAX_ABS, O_REL_RMS, errors


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


@pytest.mark.gpu
def test_two_calls_in_a_row_match_the_allocating_entry_points():
    dev = torch.device("cuda:0")
    cases = [I.custom([1000], hq=2, hkv=1, d=64, seed=2100),                  # partial last block
             I.custom([3001, 0, 257, 4096], hq=4, hkv=2, d=128, seed=2101)]   # ragged batch, other shape
    for w in cases:
        q, k, v = (t.to(dev) for t in I.draw_qkv(w))
        cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
        T = w.total_tokens
        # existing path
        route = bf1.plan_route(cu, w.max_seqlen)
        o_ref, lse_ref = bf1.attn_fwd(q, k, v, cu, w.max_seqlen, route)
        torch.cuda.synchronize()
        route.check_status()
        # new path: outputs and the status word are allocated up front, then nothing else is
        outs = [torch.full((T, w.hq, w.d), float("nan"), dtype=torch.bfloat16, device=dev) for _ in range(2)]
        lses = [torch.full((w.hq, T), float("nan"), dtype=torch.float32, device=dev) for _ in range(2)]
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated(dev)
        for rep in range(2):
            bf1.attn_fwd_noalloc(q, k, v, cu, w.max_seqlen, outs[rep], lses[rep], status=status)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated(dev) == before
        assert int(status.item()) == 0
        for rep in range(2):
            o, lse = outs[rep].float().cpu().numpy(), lses[rep].cpu().numpy()
            assert not np.isnan(o).any() and not np.isnan(lse).any()
            e = errors(o, lse, o_ref.float().cpu().numpy(), lse_ref.cpu().numpy().astype(np.float64))
            assert e["o_max_abs"] <= O_MAX_ABS and e["o_rel_rms"] <= O_REL_RMS and e["lse_max_abs"] <= LSE_ABS, (rep, e)
    # without a caller-owned status word the device status stays inside the library
    w = cases[0]
    q, k, v = (t.to(dev) for t in I.draw_qkv(w))
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
    out = torch.empty((w.total_tokens, w.hq, w.d), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((w.hq, w.total_tokens), dtype=torch.float32, device=dev)
    bf1.attn_fwd_noalloc(q, k, v, cu, w.max_seqlen, out, lse)
    route = bf1.plan_route(cu, w.max_seqlen)
    o_ref, lse_ref = bf1.attn_fwd(q, k, v, cu, w.max_seqlen, route)
    torch.cuda.synchronize()
    e = errors(out.float().cpu().numpy(), lse.cpu().numpy(), o_ref.float().cpu().numpy(),
               lse_ref.cpu().numpy().astype(np.float64))
    assert e["o_max_abs"] <= O_MAX_ABS and e["o_rel_rms"] <= O_REL_RMS and e["lse_max_abs"] <= LSE_ABS, e
