"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every symbol the
header declares, and rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

import paper_2608_20427_b200 as bf1
from paper_2608_20427_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bf1.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bf1_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = bf1.load()
    names = declared_functions()
    assert set(binding.EXPORTS) <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    assert lib.bf1_version() >= 1


def test_route_capacity_is_host_only_and_matches_the_degree_bound():
    cap, deg = bf1.route_capacity(1, 32768, 32768)
    assert cap >= 512 and deg == 11          # floor(log2 511) + 3
    cap, deg = bf1.route_capacity(4, 39922, 16384)
    assert cap >= 47 + 128 + 193 + 256 and deg == 10
    assert bf1.route_capacity(1, 1000, 1000) == (16, 6)
    assert bf1.route_capacity(1, 64, 64)[1] == 1
    assert bf1.route_capacity(1, 257, 257)[1] == 4
    # other routes
    assert bf1.route_capacity(1, 6400, 6400, bf1.RouteCfg(local_blocks=5, global_first=0, dyadic=0))[1] == 6
    assert bf1.route_capacity(1, 6400, 6400, bf1.RouteCfg(local_blocks=0, global_first=1, dyadic=0))[1] == 2


def test_bad_arguments_are_rejected_on_the_host():
    with pytest.raises(bf1.Bf1Error) as e:
        bf1.route_capacity(1, 100, 100, bf1.RouteCfg(block=32))
    assert e.value.code == -2 and "64" in str(e.value)
    with pytest.raises(bf1.Bf1Error):
        bf1.route_capacity(-1, 100, 100)
    with pytest.raises(bf1.Bf1Error):
        bf1.route_capacity(1, 100, 100, bf1.RouteCfg(local_blocks=-1))
    lib = bf1.load()
    # null tensors: refused before any CUDA call
    rc = lib.bf1_dense_causal_fwd(None, None, None, None, 1, 64, 64, 2, 1, 64, 0.0, None, None, None, None)
    assert rc == -1 and b"null" in lib.bf1_last_error()
    rc = lib.bf1_attn_fwd(None, None, None, None, 1, 64, 64, 2, 1, 64, 0.0, None, None, None, None)
    assert rc == -1
    # unsupported geometry (pointers are never dereferenced on this path)
    fake = ctypes.c_void_p(0x1000)
    for hq, hkv, d, code in ((8, 1, 64, -2), (6, 2, 64, -2), (2, 1, 96, -2), (3, 2, 64, -1)):
        rc = lib.bf1_dense_causal_fwd(fake, fake, fake, fake, 1, 64, 64, hq, hkv, d, 0.0, fake, fake, None, None)
        assert rc == code, (hq, hkv, d, lib.bf1_last_error())
    rc = lib.bf1_dense_causal_fwd(ctypes.c_void_p(0x1004), fake, fake, fake, 1, 64, 64, 2, 1, 64, 0.0, fake, fake,
                                  None, None)
    assert rc == -1 and b"aligned" in lib.bf1_last_error()
    # empty batch: OK without touching a device
    rc = lib.bf1_dense_causal_fwd(fake, fake, fake, fake, 0, 0, 0, 2, 1, 64, 0.0, fake, fake, None, None)
    assert rc == 0
