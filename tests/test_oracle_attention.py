"""Pins for the oracle's attention arithmetic (CPU only).

The paper prints no worked numeric attention example, so O and LSE are pinned by closed
forms, invariants, special cases that reduce to a library routine (torch CPU SDPA in
fp32), and brute force in pure Python on tiny inputs.
"""
import math

import numpy as np
import pytest
import torch

import bf1_inputs as I
from oracle import bf1_oracle as O


def bf(x):
    return x.to(torch.bfloat16)


def f64(t):
    return t.to(torch.float64).numpy()


def selected_count(i, b=64):
    """Columns row i attends to: b per non-self block of P(block(i)) plus the triangle part."""
    j = i // b
    if j <= 3:
        deg = j + 1
    else:
        deg = int(math.floor(math.log2(j))) + 3 - (1 if j & (j - 1) == 0 else 0)
    return b * (deg - 1) + (i % b) + 1


def brute_force(q, k, v, b, scale, W=2):
    """Pure-Python fp64 statement of the operator from Eq. 1 in generator form."""
    n, hq, d = q.shape
    hkv = k.shape[1]
    G = hq // hkv
    qq, kk, vv = f64(q), f64(k), f64(v)
    o = np.zeros((n, hq, d))
    lse = np.zeros((hq, n))
    for i in range(n):
        j = i // b
        blocks = {j - w for w in range(W + 1)} | {0}
        r = 2
        while j - 2 ** r >= 0:
            blocks.add(j - 2 ** r)
            r += 1
        cols = [c for c in range(n) if (c // b) in blocks and c <= i]
        for h in range(hq):
            s = [scale * sum(qq[i, h, t] * kk[c, h // G, t] for t in range(d)) for c in cols]
            m = max(s)
            e = [math.exp(x - m) for x in s]
            l = sum(e)
            lse[h, i] = m + math.log(l)
            for t in range(d):
                o[i, h, t] = sum(e[a] / l * vv[cols[a], h // G, t] for a in range(len(cols)))
    return o, lse


@pytest.mark.parametrize("b,n", [(1, 16), (2, 16), (4, 15), (1, 9), (2, 13)])
def test_brute_force_tiny(b, n):
    w = I.custom([n], hq=4, hkv=2, d=8, seed=100 + b * 17 + n, block=b)
    q, k, v = I.draw_qkv(w)
    c = O.cfg(block=b)
    want_o, want_lse = brute_force(q, k, v, b, 1.0 / math.sqrt(8))
    o64, l64 = O.attn_route(c, q, k, v, [0, n], fp64=True)
    np.testing.assert_allclose(o64, want_o, rtol=0, atol=1e-12)
    np.testing.assert_allclose(l64, want_lse, rtol=0, atol=1e-12)
    o32, l32 = O.attn_route(c, q, k, v, [0, n])
    np.testing.assert_allclose(o32, want_o, rtol=0, atol=2e-6)
    np.testing.assert_allclose(l32, want_lse, rtol=0, atol=2e-6)
    om, lm = O.attn_mask(q, k, v, O.token_mask(c, n), fp64=True)
    np.testing.assert_allclose(om, want_o, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lm, want_lse, rtol=0, atol=1e-12)


def test_zero_queries_give_mean_of_selected_values_and_log_count():
    n = 1000
    w = I.custom([n], hq=2, hkv=1, d=16, seed=7)
    q, k, v = I.draw_qkv(w)
    q = torch.zeros_like(q)
    c = O.cfg()
    o, lse = O.attn_route(c, q, k, v, [0, n], fp64=True)
    m = O.token_mask(c, n)
    vv = f64(v)[:, 0, :]
    for i in [0, 1, 63, 64, 255, 256, 257, 640, 999]:
        cnt = selected_count(i)
        assert m[i].sum() == cnt
        np.testing.assert_allclose(lse[:, i], math.log(cnt), atol=1e-12)
        np.testing.assert_allclose(o[i, 0], vv[m[i]].mean(axis=0), atol=1e-12)
    # fp32 form, every row
    o32, lse32 = O.attn_route(c, q, k, v, [0, n])
    want = np.log(np.array([selected_count(i) for i in range(n)], dtype=np.float64))
    np.testing.assert_allclose(lse32[0], want, atol=2e-6)


def test_constant_values_pass_through():
    n = 700
    w = I.custom([n], hq=4, hkv=2, d=32, seed=8)
    q, k, v = I.draw_qkv(w)
    const = bf(torch.arange(32, dtype=torch.float32) / 8 - 1.5)  # exactly representable
    v = const.expand(n, 2, 32).contiguous()
    o, _ = O.attn_route(O.cfg(), q, k, v, [0, n])
    np.testing.assert_allclose(o, np.broadcast_to(f64(const), o.shape), atol=1e-5)


def test_identity_values_expose_probabilities():
    """V = identity makes O the probability matrix itself: zero outside the route, rows
    sum to one, and ratios follow exp(score differences)."""
    b, n = 4, 32
    w = I.custom([n], hq=2, hkv=2, d=n, seed=9, block=b)
    q, k, _ = I.draw_qkv(w)
    v = bf(torch.eye(n)).reshape(n, 1, n).expand(n, 2, n).contiguous()
    c = O.cfg(block=b)
    o, lse = O.attn_route(c, q, k, v, [0, n], fp64=True)
    m = O.token_mask(c, n)
    scale = 1.0 / math.sqrt(n)
    for h in range(2):
        p = o[:, h, :]
        assert (p[~m] == 0).all() and (p[m] > 0).all()
        np.testing.assert_allclose(p.sum(axis=1), 1.0, atol=1e-12)
        s = scale * f64(q)[:, h, :] @ f64(k)[:, h, :].T
        np.testing.assert_allclose(p[m], np.exp(s - lse[h][:, None])[m], rtol=1e-10)


def test_single_token():
    w = I.custom([1], hq=2, hkv=1, d=64, seed=10)
    q, k, v = I.draw_qkv(w)
    o, lse = O.attn_route(O.cfg(), q, k, v, [0, 1], fp64=True)
    np.testing.assert_allclose(o[0, 0], f64(v)[0, 0], atol=0)
    np.testing.assert_allclose(o[0, 1], f64(v)[0, 0], atol=0)
    want = (f64(q)[0] @ f64(k)[0, 0]) / 8.0
    np.testing.assert_allclose(lse[:, 0], want, atol=1e-12)


@pytest.mark.parametrize("n", [1, 63, 64, 65, 192, 256])
def test_short_sequences_equal_dense_causal_bitwise(n):
    w = I.custom([n], hq=4, hkv=2, d=64, seed=11 + n)
    q, k, v = I.draw_qkv(w)
    o1, l1 = O.attn_route(O.cfg(), q, k, v, [0, n])
    o2, l2 = O.dense_causal(q, k, v, [0, n])
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)


def sdpa(q, k, v, mask=None):
    """torch CPU fp32 scaled_dot_product_attention on [n, h, d] inputs (library routine)."""
    qq, kk, vv = (x.to(torch.float32).transpose(0, 1).unsqueeze(0) for x in (q, k, v))
    if mask is None:
        out = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv, is_causal=True, enable_gqa=True)
    else:
        out = torch.nn.functional.scaled_dot_product_attention(
            qq, kk, vv, attn_mask=torch.from_numpy(mask)[None, None], enable_gqa=True)
    return out[0].transpose(0, 1).numpy()


def test_dense_causal_matches_library_sdpa_with_grouped_heads():
    n = 300
    w = I.custom([n], hq=8, hkv=2, d=64, seed=12)   # G = 4, distinct K/V per KV head
    q, k, v = I.draw_qkv(w)
    o, lse = O.dense_causal(q, k, v, [0, n])
    np.testing.assert_allclose(o, sdpa(q, k, v), atol=2e-5)
    # LSE against a direct fp64 evaluation
    G = 4
    for h in (0, 3, 4, 7):
        s = (f64(q)[:, h] @ f64(k)[:, h // G].T) / 8.0
        s[np.triu_indices(n, 1)] = -np.inf
        want = np.log(np.exp(s - s.max(axis=1, keepdims=True)).sum(axis=1)) + s.max(axis=1)
        np.testing.assert_allclose(lse[h], want, atol=3e-6)


@pytest.mark.parametrize("n,hq,hkv,d", [(1000, 2, 1, 64), (777, 16, 8, 128)])
def test_routed_attention_matches_library_sdpa_under_the_route_mask(n, hq, hkv, d):
    w = I.custom([n], hq=hq, hkv=hkv, d=d, seed=13, sink_scale=4.0)
    q, k, v = I.draw_qkv(w)
    c = O.cfg()
    m = O.token_mask(c, n)
    o_def, l_def = O.attn_mask(q, k, v, m)
    np.testing.assert_allclose(o_def, sdpa(q, k, v, m), atol=2e-5)
    # block-skipping form is the defining form, bit for bit
    o_skip, l_skip = O.attn_route(c, q, k, v, [0, n])
    assert np.array_equal(o_def, o_skip) and np.array_equal(l_def, l_skip)


def test_fp32_rounding_noise_is_far_below_the_parity_tolerance():
    w = I.WORKLOADS["tiny"]
    q, k, v = I.draw_qkv(w)
    o32, l32 = O.attn_route(O.cfg(), q, k, v, w.cu_seqlens())
    o64, l64 = O.attn_route(O.cfg(), q, k, v, w.cu_seqlens(), fp64=True)
    assert np.abs(o32 - o64).max() < 1e-5
    assert np.abs(l32 - l64).max() < 1e-5


def test_future_token_isolation_is_bitwise():
    w = I.custom([600], hq=4, hkv=2, d=64, seed=14)
    q, k, v = I.draw_qkv(w)
    c = O.cfg()
    o, lse = O.attn_route(c, q, k, v, [0, 600])
    for t in (0, 63, 64, 300, 598):
        q2, k2, v2 = I.mutate_after(w, q, k, v, 0, t, seed=99 + t)
        assert not torch.equal(k2, k)
        o2, lse2 = O.attn_route(c, q2, k2, v2, [0, 600])
        assert np.array_equal(o[:t + 1], o2[:t + 1])
        assert np.array_equal(lse[:, :t + 1], lse2[:, :t + 1])
        assert not np.array_equal(o[t + 1:], o2[t + 1:])


def test_packed_batch_equals_per_sequence_runs_bitwise():
    lens = [130, 0, 257, 64, 1]
    w = I.custom(lens, hq=4, hkv=2, d=64, seed=15)
    q, k, v = I.draw_qkv(w)
    cu = w.cu_seqlens()
    c = O.cfg()
    o, lse = O.attn_route(c, q, k, v, cu)
    od, lsed = O.dense_causal(q, k, v, cu)
    assert not np.isnan(o).any() and not np.isnan(lse).any()
    for s, n in enumerate(lens):
        if n == 0:
            continue
        sl = slice(cu[s], cu[s + 1])
        o1, l1 = O.attn_route(c, q[sl], k[sl], v[sl], [0, n])
        assert np.array_equal(o[sl], o1) and np.array_equal(lse[:, sl], l1)
        o2, l2 = O.dense_causal(q[sl], k[sl], v[sl], [0, n])
        assert np.array_equal(od[sl], o2) and np.array_equal(lsed[:, sl], l2)


def test_row_sampling_fills_only_the_requested_rows():
    w = I.custom([500, 300], hq=2, hkv=1, d=64, seed=16)
    q, k, v = I.draw_qkv(w)
    cu = w.cu_seqlens()
    full_o, full_l = O.attn_route(O.cfg(), q, k, v, cu)
    rows = [0, 63, 64, 499, 500, 501, 799]
    o, lse = O.attn_route(O.cfg(), q, k, v, cu, rows=rows)
    assert np.array_equal(o[rows], full_o[rows]) and np.array_equal(lse[:, rows], full_l[:, rows])
    rest = np.setdiff1d(np.arange(800), rows)
    assert np.isnan(o[rest]).all() and np.isnan(lse[:, rest]).all()
    d_o, d_l = O.dense_causal(q, k, v, cu, rows=rows)
    f_o, f_l = O.dense_causal(q, k, v, cu)
    assert np.array_equal(d_o[rows], f_o[rows]) and np.array_equal(d_l[:, rows], f_l[:, rows])


def test_head_permutation_permutes_outputs():
    n = 400
    w = I.custom([n], hq=4, hkv=2, d=64, seed=17)
    q, k, v = I.draw_qkv(w)
    o, lse = O.attn_route(O.cfg(), q, k, v, [0, n])
    # swap the two KV groups (query heads 0,1 <-> 2,3 and KV heads 0 <-> 1)
    qp = q[:, [2, 3, 0, 1]].contiguous()
    kp, vp = k[:, [1, 0]].contiguous(), v[:, [1, 0]].contiguous()
    o2, lse2 = O.attn_route(O.cfg(), qp, kp, vp, [0, n])
    assert np.array_equal(o[:, [2, 3, 0, 1]], o2) and np.array_equal(lse[[2, 3, 0, 1]], lse2)
    # swapping query heads inside a group only permutes those outputs
    qs = q[:, [1, 0, 2, 3]].contiguous()
    o3, _ = O.attn_route(O.cfg(), qs, k, v, [0, n])
    assert np.array_equal(o[:, [1, 0, 2, 3]], o3)


def test_scale_argument():
    n = 200
    w = I.custom([n], hq=2, hkv=1, d=64, seed=18)
    q, k, v = I.draw_qkv(w)
    o_def, _ = O.attn_route(O.cfg(), q, k, v, [0, n])
    o_same, _ = O.attn_route(O.cfg(), q, k, v, [0, n], scale=0.125)
    assert np.array_equal(o_def, o_same)
    o_hot, l_hot = O.attn_route(O.cfg(), q, k, v, [0, n], scale=0.5, fp64=True)
    qq, kk = f64(q)[:, 0], f64(k)[:, 0]
    s = 0.5 * qq @ kk.T
    s[np.triu_indices(n, 1)] = -np.inf
    want = np.log(np.exp(s - s.max(axis=1, keepdims=True)).sum(axis=1)) + s.max(axis=1)
    np.testing.assert_allclose(l_hot[0], want, atol=1e-10)
