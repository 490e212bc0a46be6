"""Pins for the oracle's route, mask and selected-pair accounting (CPU only).

Each test ties the oracle to something other than itself: a value the paper prints, a
closed form, an independent enumeration of Eq. 1 in generator form, or a hand drawing.
"""
import math
import os
import re

import numpy as np
import pytest

from oracle import bf1_oracle as O

from conftest import GOLDEN, read_golden

PAPER = read_golden("paper_values.txt")


def paper(key, typ=float):
    return typ(PAPER[key][0])


def generator_P(j, W=2, global_first=True, dyadic=True, r_min=2):
    """Eq. 1 as a set builder, written independently of the oracle's predicate:
    {j, j-1, ..., j-W, 0} u {j - 2^r : r >= r_min}, invalid indices dropped."""
    s = {j - w for w in range(W + 1)}
    if global_first:
        s.add(0)
    if dyadic:
        r = r_min
        while j - (1 << r) >= 0:
            s.add(j - (1 << r))
            r += 1
    return sorted(x for x in s if x >= 0)


def degree_closed_form(j):
    if j <= 3:
        return j + 1
    return int(math.floor(math.log2(j))) + 3 - (1 if j & (j - 1) == 0 else 0)


def S_closed(B):
    """Selected block pairs for B blocks."""
    if B == 1:
        return 1
    L = int(math.floor(math.log2(B - 1)))
    return B * (L + 3) - 2 ** (L + 1) - L - 1


def T_closed(n, b=64):
    """Selected token pairs for n tokens (triangle on the self block)."""
    B = (n + b - 1) // b
    r = n - (B - 1) * b
    full = 0
    if B > 1:
        full = b * b * (S_closed(B - 1) - (B - 1)) + (B - 1) * b * (b + 1) // 2
    return full + r * b * (degree_closed_form(B - 1) - 1) + r * (r + 1) // 2


def test_reported_configuration_matches_paper():
    c = O.cfg()
    assert c.block == paper("block_width", int)
    assert c.local_blocks == paper("local_predecessor_blocks", int)
    # first dyadic offset that is not already a local block is 4 = 2^2 (Eq. 1, r >= 2)
    j = 100
    non_local = [j - p for p in generator_P(j) if j - p > c.local_blocks and p != 0]
    assert min(non_local) == paper("dyadic_first_offset_blocks", int)


def test_interaction_reduction_32k_matches_table2():
    """Table 2 / Section 5.1: 26.98x fewer selected interactions than dense causal at 32K."""
    n = 32768
    _, _, _, total = O.route(O.cfg(), n)
    dense = n * (n + 1) // 2
    assert round(dense / total, 2) == paper("interaction_reduction_32k")
    assert total == 19_902_464
    # the pin is sharp: the nearby readings of the route all miss the printed value
    for alt in (O.cfg(global_first=0), O.cfg(local_blocks=3), O.cfg(local_blocks=1, dyadic=0),
                O.cfg(dyadic=0)):
        _, _, _, t_alt = O.route(alt, n)
        assert round(dense / t_alt, 2) != paper("interaction_reduction_32k")
    # ... and so do the other ways of counting the self block (full tile instead of triangle)
    idx, cnt, _, _ = O.route(O.cfg(), n)
    full_diag = int(sum(64 * 64 * int(x) for x in cnt))
    assert round(dense / full_diag, 2) != paper("interaction_reduction_32k")


def test_max_shortest_path_matches_prop2():
    c = O.cfg()
    assert O.max_shortest_path(c, 512) == paper("max_shortest_path_B512", int)
    assert O.max_shortest_path(c, 32768 // c.block) == paper("hops_32k", int)
    # popcount bound of the proof: path length <= popcount(delta) <= floor(log2 B)
    for B in (8, 16, 64, 128):
        assert O.max_shortest_path(c, B) <= int(math.log2(B))
    # without the dyadic edges the graph is a width-2 window plus block 0: depth grows linearly
    assert O.max_shortest_path(O.cfg(dyadic=0), 64) > 8


def test_degree_bound_of_prop1():
    c = O.cfg()
    bm = O.block_mask(c, 3000 * c.block)
    deg = bm.sum(axis=1)
    const = paper("degree_bound_constant", int)
    for j in range(1, len(deg)):
        assert deg[j] <= const + int(math.floor(math.log2(j)))
        assert deg[j] == degree_closed_form(j)
    assert deg[0] == 1


def test_predicate_equals_generator_form():
    c = O.cfg(block=1)
    n = 2000
    bm = O.block_mask(c, n)
    for j in range(n):
        assert list(np.nonzero(bm[j])[0]) == generator_P(j), j
    # the "every k >= 0" reading and Eq. 1's "r >= 2" coincide when W = 2 ...
    for j in range(300):
        assert generator_P(j, r_min=0) == generator_P(j, r_min=2)
    # ... and the knobs act independently
    bm0 = O.block_mask(O.cfg(block=1, local_blocks=0), 300)
    for j in range(300):
        assert list(np.nonzero(bm0[j])[0]) == generator_P(j, W=0, r_min=0)
    bm1 = O.block_mask(O.cfg(block=1, global_first=0, dyadic=0, local_blocks=3), 50)
    for j in range(50):
        assert list(np.nonzero(bm1[j])[0]) == [x for x in range(j - 3, j + 1) if x >= 0]


def test_token_mask_equals_hand_drawing():
    rows = []
    with open(os.path.join(GOLDEN, "eq1_b1_n16.txt")) as f:
        for line in f:
            line = line.rstrip("\n")
            if re.fullmatch(r"[#.]{16}", line):
                rows.append([ch == "#" for ch in line])
    want = np.array(rows, dtype=bool)
    assert want.shape == (16, 16)
    got = O.token_mask(O.cfg(block=1), 16)
    assert (got == want).all()


def test_token_mask_structure():
    """Self block: causal triangle.  Other selected blocks: full and strictly earlier."""
    c = O.cfg(block=4)
    n = 4 * 21 + 3  # partial last block
    m = O.token_mask(c, n)
    bm = O.block_mask(c, n)
    B = bm.shape[0]
    assert not np.triu(m, 1).any()  # no future column anywhere
    for jq in range(B):
        r0, r1 = 4 * jq, min(4 * jq + 4, n)
        for jk in range(B):
            c0, c1 = 4 * jk, min(4 * jk + 4, n)
            tile = m[r0:r1, c0:c1]
            if jk == jq:
                assert (tile == np.tril(np.ones_like(tile))).all()
            elif bm[jq, jk]:
                assert jk < jq and tile.all()
            else:
                assert not tile.any()


@pytest.mark.parametrize("b", [64, 128])
def test_token_mask_at_both_block_widths_equals_eq1_token_by_token(b):
    """The block width is a parameter of the method: token i (block i // b) sees token c (block c // b)
    iff c <= i and c's block is in P(i's block), Eq. 1 written out per token pair."""
    n = 5 * 128 + 70   # a partial last block at either width
    got = O.token_mask(O.cfg(block=b), n)
    want = np.zeros((n, n), dtype=bool)
    for i in range(n):
        sel = set(generator_P(i // b))
        for c in range(i + 1):
            want[i, c] = (c // b) in sel
    assert (got == want).all()
    _, cnt, pairs, total = O.route(O.cfg(block=b), n)
    assert total == int(want.sum()) == int(pairs.sum())
    assert [int(x) for x in cnt] == [len(generator_P(j)) for j in range((n + b - 1) // b)]


def test_closed_form_totals_all_lengths():
    c = O.cfg()
    for n in list(range(1, 4097, 7)) + [64, 128, 192, 193, 256, 257, 1000, 4096]:
        idx, cnt, pc, total = O.route(c, n)
        B = (n + 63) // 64
        assert len(cnt) == B
        assert int(cnt.sum()) == S_closed(B), n
        assert total == T_closed(n), n
        assert total == int(pc.sum())
        assert total == int(O.token_mask(c, n).sum()) if n <= 1024 else True


def test_n_log_n_total_for_power_of_two_lengths():
    b = 64
    for m in range(0, 10):
        n = b << m
        _, cnt, _, total = O.route(O.cfg(), n)
        assert int(cnt.sum()) == (m + 1) * 2 ** m - m
        assert total == n * b * m - b * b * m + n * (b + 1) // 2


def test_route_lists_are_sorted_unique_and_end_with_self():
    c = O.cfg()
    n = 12345
    idx, cnt, pc, total = O.route(c, n, max_deg=16)
    for j in range(len(cnt)):
        lst = idx[j, :cnt[j]]
        assert list(lst) == generator_P(j)
        assert (idx[j, cnt[j]:] == -1).all()
        assert lst[-1] == j and (np.diff(lst) > 0).all()
        rows = min(64, n - 64 * j)
        assert pc[j] == rows * 64 * (cnt[j] - 1) + rows * (rows + 1) // 2
    with pytest.raises(ValueError):
        O.route(c, n, max_deg=5)


def test_length_257_differs_from_dense_in_one_row():
    """Partial final block gate (Section 4.2): at 257 tokens block 4 holds one token and
    skips block 1 only, so the mask differs from plain causal in row 256, columns 64..127."""
    m = O.token_mask(O.cfg(), 257)
    dense = np.tril(np.ones((257, 257), dtype=bool))
    diff = dense & ~m
    assert not (m & ~dense).any()
    assert diff.sum() == 64
    assert diff[256, 64:128].all()


def test_short_sequences_are_dense():
    """For j <= 3 the route selects every predecessor, so n <= 4b is plain causal."""
    for n in (1, 63, 64, 65, 192, 256):
        assert (O.token_mask(O.cfg(), n) == np.tril(np.ones((n, n), dtype=bool))).all()
    n = 321
    assert not (O.token_mask(O.cfg(), n) == np.tril(np.ones((n, n), dtype=bool))).all()


def test_stored_counts_for_the_workloads():
    """tests/golden/route_counts.txt is written by make_golden.py from the oracle; the
    closed forms above re-derive every entry, so a stale file is caught here."""
    stored = read_golden("route_counts.txt")
    for key, (val, _) in stored.items():
        n = int(key.split("_")[1])
        blocks, pairs, tokens = (int(x) for x in val.split())
        B = (n + 63) // 64
        assert blocks == B and pairs == S_closed(B) and tokens == T_closed(n)
        _, cnt, _, total = O.route(O.cfg(), n)
        assert (len(cnt), int(cnt.sum()), total) == (blocks, pairs, tokens)
