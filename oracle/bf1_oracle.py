"""ctypes wrapper around the BF1 CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Only tests, the smoke check and the benchmark's cpu-baseline leg may import this module;
the CUDA package never does.  The wrapper only marshals arguments: all arithmetic is in
``bf1_oracle.c`` / ``bf1_oracle_attn.inc`` beside this file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = [os.path.join(_HERE, "bf1_oracle.c"), os.path.join(_HERE, "bf1_oracle_attn.inc")]
_LIB_PATH = os.path.join(_HERE, "libbf1_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its source."""
    stale = force or not os.path.exists(_LIB_PATH) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB_PATH) for s in _SRC)
    if stale:
        tmp = _LIB_PATH + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp",
               "-fno-fast-math", "-ffp-contract=off", "-o", tmp, _SRC[0], "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


class Cfg(ctypes.Structure):
    _fields_ = [("block", ctypes.c_int32), ("local_blocks", ctypes.c_int32),
                ("global_first", ctypes.c_int32), ("dyadic", ctypes.c_int32)]


def cfg(block: int = 64, local_blocks: int = 2, global_first: int = 1, dyadic: int = 1) -> Cfg:
    return Cfg(block, local_blocks, global_first, dyadic)


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i32, i64, f64, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        cp = ctypes.POINTER(Cfg)
        L.bf1o_sel.restype = ctypes.c_int
        L.bf1o_sel.argtypes = [cp, i64, i64]
        L.bf1o_num_blocks.restype = i64
        L.bf1o_num_blocks.argtypes = [cp, i64]
        L.bf1o_route.restype = i64
        L.bf1o_route.argtypes = [cp, i64, i32, vp, vp, vp]
        L.bf1o_block_mask.restype = None
        L.bf1o_block_mask.argtypes = [cp, i64, vp]
        L.bf1o_token_mask.restype = None
        L.bf1o_token_mask.argtypes = [cp, i64, vp]
        L.bf1o_max_shortest_path.restype = i32
        L.bf1o_max_shortest_path.argtypes = [cp, i32]
        L.bf1o_threads.restype = ctypes.c_int
        for suf in ("_f32", "_f64"):
            f = getattr(L, "bf1o_attn_mask" + suf)
            f.restype = None
            f.argtypes = [vp, vp, vp, i64, i32, i32, i32, f64, vp, vp, vp]
            f = getattr(L, "bf1o_attn_route" + suf)
            f.restype = None
            f.argtypes = [cp, vp, vp, vp, vp, i32, i32, i32, i32, f64, vp, i64, vp, vp]
            f = getattr(L, "bf1o_attn_route_bwd" + suf)
            f.restype = None
            f.argtypes = [cp, vp, vp, vp, vp, vp, i32, i32, i32, i32, f64, vp, vp, vp]
            f = getattr(L, "bf1o_dense_causal" + suf)
            f.restype = None
            f.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, f64, vp, i64, vp, vp]
        _lib = L
    return _lib


def threads() -> int:
    return int(lib().bf1o_threads())


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def bf16_bits(t) -> np.ndarray:
    """Raw bf16 bit patterns of a CPU torch bf16 tensor, as a contiguous uint16 array."""
    import torch
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return np.ascontiguousarray(t.contiguous().view(torch.int16).numpy()).view(np.uint16)


def sel(c: Cfg, jq: int, jk: int) -> bool:
    return bool(lib().bf1o_sel(ctypes.byref(c), jq, jk))


def max_degree(c: Cfg, n: int) -> int:
    """Largest |P(j)| over the blocks of a sequence of n tokens (by enumeration)."""
    B = int(lib().bf1o_num_blocks(ctypes.byref(c), n))
    best = 1
    for jq in range(B):
        best = max(best, sum(1 for jk in range(jq + 1) if lib().bf1o_sel(ctypes.byref(c), jq, jk)))
    return best


def route(c: Cfg, n: int, max_deg: Optional[int] = None):
    """(kv_idx [B, max_deg] int32 with -1 padding, kv_count [B], pair_count [B] int64, total)."""
    B = int(lib().bf1o_num_blocks(ctypes.byref(c), n))
    if max_deg is None:
        max_deg = B  # always enough
    kv_idx = np.full((B, max_deg), -1, dtype=np.int32)
    kv_count = np.zeros((B,), dtype=np.int32)
    pair_count = np.zeros((B,), dtype=np.int64)
    total = lib().bf1o_route(ctypes.byref(c), n, max_deg, _ptr(kv_idx), _ptr(kv_count), _ptr(pair_count))
    if total < 0:
        raise ValueError("max_degree too small")
    return kv_idx, kv_count, pair_count, int(total)


def block_mask(c: Cfg, n: int) -> np.ndarray:
    B = int(lib().bf1o_num_blocks(ctypes.byref(c), n))
    bm = np.zeros((B, B), dtype=np.uint8)
    lib().bf1o_block_mask(ctypes.byref(c), n, _ptr(bm))
    return bm.astype(bool)


def token_mask(c: Cfg, n: int) -> np.ndarray:
    m = np.zeros((n, n), dtype=np.uint8)
    lib().bf1o_token_mask(ctypes.byref(c), n, _ptr(m))
    return m.astype(bool)


def max_shortest_path(c: Cfg, num_blocks: int) -> int:
    return int(lib().bf1o_max_shortest_path(ctypes.byref(c), num_blocks))


def _out(T: int, hq: int, d: int, dtype):
    # NaN-filled so that an unwritten row cannot pass for a result
    return (np.full((T, hq, d), np.nan, dtype=dtype), np.full((hq, T), np.nan, dtype=dtype))


def _scale(scale: Optional[float], d: int) -> float:
    return float(scale) if scale is not None and scale > 0 else 1.0 / float(np.sqrt(d))


def attn_mask(q, k, v, mask: np.ndarray, scale: Optional[float] = None, fp64: bool = False):
    """Defining form, one sequence: masked softmax attention under an explicit n x n mask.
    q [n, hq, d], k/v [n, hkv, d] torch bf16.  Returns (O [n, hq, d], LSE [hq, n])."""
    n, hq, d = q.shape
    hkv = k.shape[1]
    dtype = np.float64 if fp64 else np.float32
    o, lse = _out(n, hq, d, dtype)
    m8 = np.ascontiguousarray(mask.astype(np.uint8))
    qb, kb, vb = bf16_bits(q), bf16_bits(k), bf16_bits(v)
    f = lib().bf1o_attn_mask_f64 if fp64 else lib().bf1o_attn_mask_f32
    f(_ptr(qb), _ptr(kb), _ptr(vb), n, hq, hkv, d, _scale(scale, d), _ptr(m8), _ptr(o), _ptr(lse))
    return o, lse


def attn_route(c: Cfg, q, k, v, cu_seqlens: Sequence[int], scale: Optional[float] = None,
               rows: Optional[Sequence[int]] = None, fp64: bool = False):
    """Block-skipping form over a packed batch.  ``rows``: optional global token rows to
    compute (others stay NaN)."""
    T, hq, d = q.shape
    hkv = k.shape[1]
    dtype = np.float64 if fp64 else np.float32
    o, lse = _out(T, hq, d, dtype)
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
    assert cu[-1] == T
    qb, kb, vb = bf16_bits(q), bf16_bits(k), bf16_bits(v)
    if rows is None:
        rp, nr = None, 0
    else:
        ra = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
        rp, nr = _ptr(ra), len(ra)
    f = lib().bf1o_attn_route_f64 if fp64 else lib().bf1o_attn_route_f32
    f(ctypes.byref(c), _ptr(qb), _ptr(kb), _ptr(vb), _ptr(cu), len(cu) - 1, hq, hkv, d,
      _scale(scale, d), rp, nr, _ptr(o), _ptr(lse))
    return o, lse


def dense_causal(q, k, v, cu_seqlens: Sequence[int], scale: Optional[float] = None,
                 rows: Optional[Sequence[int]] = None, fp64: bool = False):
    """Plain causal attention over a packed batch (the dense comparator)."""
    T, hq, d = q.shape
    hkv = k.shape[1]
    dtype = np.float64 if fp64 else np.float32
    o, lse = _out(T, hq, d, dtype)
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
    assert cu[-1] == T
    qb, kb, vb = bf16_bits(q), bf16_bits(k), bf16_bits(v)
    if rows is None:
        rp, nr = None, 0
    else:
        ra = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
        rp, nr = _ptr(ra), len(ra)
    f = lib().bf1o_dense_causal_f64 if fp64 else lib().bf1o_dense_causal_f32
    f(_ptr(qb), _ptr(kb), _ptr(vb), _ptr(cu), len(cu) - 1, hq, hkv, d, _scale(scale, d),
      rp, nr, _ptr(o), _ptr(lse))
    return o, lse


def attn_route_bwd(c: Cfg, q, k, v, d_o: np.ndarray, cu_seqlens: Sequence[int], scale: Optional[float] = None,
                   fp64: bool = True):
    """Gradients (dq, dk, dv) of the routed attention for an upstream gradient d_o [T, hq, d]."""
    T, hq, d = q.shape
    hkv = k.shape[1]
    dtype = np.float64 if fp64 else np.float32
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
    qb, kb, vb = bf16_bits(q), bf16_bits(k), bf16_bits(v)
    go = np.ascontiguousarray(d_o.astype(dtype))
    dq = np.empty((T, hq, d), dtype=dtype)
    dk = np.empty((T, hkv, d), dtype=dtype)
    dv = np.empty((T, hkv, d), dtype=dtype)
    f = lib().bf1o_attn_route_bwd_f64 if fp64 else lib().bf1o_attn_route_bwd_f32
    f(ctypes.byref(c), _ptr(qb), _ptr(kb), _ptr(vb), _ptr(go), _ptr(cu), len(cu) - 1, hq, hkv, d,
      _scale(scale, d), _ptr(dq), _ptr(dk), _ptr(dv))
    return dq, dk, dv
