"""Pins for the oracle's gradients (CPU only): library autograd through SDPA under the route's
boolean mask, central finite differences of the oracle's own forward, and causality of gradients."""
import numpy as np
import torch

import bf1_inputs as I
from oracle import bf1_oracle as O


def autograd_reference(q, k, v, mask, d_o):
    """torch CPU fp64 autograd through scaled_dot_product_attention with the boolean mask."""
    qq = q.to(torch.float64).transpose(0, 1).unsqueeze(0).requires_grad_(True)
    kk = k.to(torch.float64).transpose(0, 1).unsqueeze(0).requires_grad_(True)
    vv = v.to(torch.float64).transpose(0, 1).unsqueeze(0).requires_grad_(True)
    out = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv, attn_mask=torch.from_numpy(mask)[None, None],
                                                           enable_gqa=True)
    out.backward(torch.from_numpy(d_o).transpose(0, 1).unsqueeze(0))
    back = lambda t: t.grad[0].transpose(0, 1).numpy()
    return back(qq), back(kk), back(vv)


def test_gradients_match_library_autograd_under_the_route_mask():
    n = 333                                             # 6 blocks, partial last one, route differs from dense
    w = I.custom([n], hq=4, hkv=2, d=32, seed=5000)
    q, k, v = I.draw_qkv(w)
    rng = np.random.default_rng(0)
    d_o = rng.standard_normal((n, 4, 32))
    c = O.cfg()
    dq, dk, dv = O.attn_route_bwd(c, q, k, v, d_o, [0, n])
    rq, rk, rv = autograd_reference(q, k, v, O.token_mask(c, n), d_o)
    np.testing.assert_allclose(dq, rq, atol=1e-10)
    np.testing.assert_allclose(dk, rk, atol=1e-10)
    np.testing.assert_allclose(dv, rv, atol=1e-10)
    # fp32 instantiation stays close
    dq32, dk32, dv32 = O.attn_route_bwd(c, q, k, v, d_o, [0, n], fp64=False)
    assert max(np.abs(dq32 - rq).max(), np.abs(dk32 - rk).max(), np.abs(dv32 - rv).max()) < 2e-4


def test_gradients_match_finite_differences_of_the_forward():
    b, n = 2, 11
    w = I.custom([n], hq=2, hkv=1, d=8, seed=5001, block=b)
    q, k, v = I.draw_qkv(w)
    c = O.cfg(block=b)
    rng = np.random.default_rng(1)
    d_o = rng.standard_normal((n, 2, 8))
    dq, dk, dv = O.attn_route_bwd(c, q, k, v, d_o, [0, n])

    def loss(qq, kk, vv):
        o, _ = O.attn_route(c, qq, kk, vv, [0, n], fp64=True)
        return float((o * d_o).sum())

    # bf16 inputs: step by a representable amount (2^-5 on values of size ~1), central differences
    for name, grad in (("q", dq), ("k", dk), ("v", dv)):
        for idx in [(0, 0, 0), (5, 0, 3), (10, 0, 7), (7, 0, 1)]:
            base = {"q": q, "k": k, "v": v}
            t = base[name].clone().float()
            h = 2.0 ** -5
            tp, tm = t.clone(), t.clone()
            tp[idx] = torch.tensor(float(t[idx]) + h).to(torch.bfloat16).float()
            tm[idx] = torch.tensor(float(t[idx]) - h).to(torch.bfloat16).float()
            step = float(tp[idx] - tm[idx])
            args_p = dict(base); args_p[name] = tp.to(torch.bfloat16)
            args_m = dict(base); args_m[name] = tm.to(torch.bfloat16)
            fd = (loss(args_p["q"], args_p["k"], args_p["v"]) - loss(args_m["q"], args_m["k"], args_m["v"])) / step
            assert abs(fd - grad[idx]) < 5e-3 * max(1.0, abs(grad[idx])), (name, idx, fd, grad[idx])


def test_gradients_respect_causality_and_the_route():
    n = 400
    w = I.custom([n, 70], hq=4, hkv=2, d=16, seed=5002)
    q, k, v = I.draw_qkv(w)
    c = O.cfg()
    T = n + 70
    d_o = np.zeros((T, 4, 16))
    t = 300                                            # upstream gradient only on row t of sequence 0
    d_o[t] = 1.0
    dq, dk, dv = O.attn_route_bwd(c, q, k, v, d_o, w.cu_seqlens())
    sel = O.token_mask(c, n)[t]                         # columns row t attends to
    assert (np.abs(dq[np.arange(T) != t]) == 0).all() and np.abs(dq[t]).max() > 0
    assert (np.abs(dk[:n][~sel]) == 0).all() and (np.abs(dv[:n][~sel]) == 0).all()
    assert (np.abs(dv[:n][sel]).max(axis=(1, 2)) > 0).all()
    assert (dk[n:] == 0).all() and (dv[n:] == 0).all()  # the other sequence is untouched
    assert np.isfinite(dq).all() and np.isfinite(dk).all() and np.isfinite(dv).all()
