"""Seeded synthetic inputs for the BF1 forward operator.

This module is the only code shared by the CPU oracle's tests and the CUDA path's
tests/bench.  It holds none of the method's arithmetic: it only names the workload
configurations and draws Q, K, V.

The paper evaluates the operator inside Qwen3-0.6B (16 query heads, 8 KV heads, head
dimension 128, block width 64, batch 1; Section 4.1, Section 3.1) on a private
question-answer corpus.  Neither weights nor corpus are needed for an operator whose
cost depends only on shapes and the route, so every input here is i.i.d. N(0,1) drawn
on the CPU with a fixed seed and rounded to bf16; the same bf16 bytes are given to the
oracle and to the GPU.  Draw order is Q, then K, then V.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import torch


@dataclass(frozen=True)
class Workload:
    """One synthetic workload: a packed batch of sequences in one attention geometry."""
    name: str
    seqlens: Tuple[int, ...]
    hq: int
    hkv: int
    d: int
    seed: int
    sink_scale: float = 1.0        # K row 0 of every sequence is multiplied by this
    block: int = 64
    local_blocks: int = 2
    global_first: int = 1
    dyadic: int = 1

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seqlens))

    @property
    def batch(self) -> int:
        return len(self.seqlens)

    @property
    def max_seqlen(self) -> int:
        return max(self.seqlens) if self.seqlens else 0

    def cu_seqlens(self) -> List[int]:
        out = [0]
        for n in self.seqlens:
            out.append(out[-1] + int(n))
        return out


def _qwen(name: str, seqlens, seed: int, sink_scale: float = 1.0) -> Workload:
    return Workload(name=name, seqlens=tuple(seqlens), hq=16, hkv=8, d=128, seed=seed,
                    sink_scale=sink_scale)


# The five benchmark configurations (tiny / 4K with a sink row / length sweep / 32K /
# ragged batch).  "layers" for the 32K point are produced by seed + layer index.
WORKLOADS = {
    "tiny": Workload(name="tiny", seqlens=(1000,), hq=2, hkv=1, d=64, seed=1001),
    "qwen_4k": _qwen("qwen_4k", (4096,), 4096, sink_scale=4.0),
    "qwen_2k": _qwen("qwen_2k", (2048,), 2048),
    "qwen_8k": _qwen("qwen_8k", (8192,), 8192),
    "qwen_16k": _qwen("qwen_16k", (16384,), 16384),
    "qwen_32k": _qwen("qwen_32k", (32768,), 32768),
    "ragged": _qwen("ragged", (3001, 8192, 12345, 16384), 5005),
}


def custom(seqlens, hq: int, hkv: int, d: int, seed: int, sink_scale: float = 1.0,
           **route) -> Workload:
    """A workload outside the named list (unit-test sizes)."""
    return Workload(name="custom", seqlens=tuple(int(x) for x in seqlens), hq=hq, hkv=hkv,
                    d=d, seed=seed, sink_scale=sink_scale, **route)


def draw_qkv(w: Workload, layer: int = 0):
    """Return (q, k, v) as CPU bf16 tensors of shape [T, hq, d], [T, hkv, d], [T, hkv, d].

    Values are N(0,1) in fp32 from a CPU generator seeded with ``w.seed + layer``; K row 0
    of each sequence is scaled by ``w.sink_scale`` before the cast to bf16.
    """
    g = torch.Generator(device="cpu")
    g.manual_seed(int(w.seed) + int(layer))
    t = w.total_tokens
    q = torch.randn((t, w.hq, w.d), generator=g, dtype=torch.float32)
    k = torch.randn((t, w.hkv, w.d), generator=g, dtype=torch.float32)
    v = torch.randn((t, w.hkv, w.d), generator=g, dtype=torch.float32)
    if w.sink_scale != 1.0:
        cu = w.cu_seqlens()
        for s in range(w.batch):
            if w.seqlens[s] > 0:
                k[cu[s]] *= w.sink_scale
    return q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)


def static_random_lists(num_blocks: int, seed: int, local_blocks: int = 2):
    """A fixed random non-local block graph with the BF1 route's per-block list lengths: for query
    block j the list is j itself plus a seeded random subset of its predecessors, as many as the
    paper's route reads for that block (Section 4.3's static-random control; the paper does not give
    its construction, so this one is this repository's own).  Returns one ascending list per block,
    self block last.  Pure index bookkeeping: no attention arithmetic."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    lists = []
    for j in range(num_blocks):
        want = {j, 0} | {j - w for w in range(1, local_blocks + 1) if j - w >= 0}
        k = 0
        while j - (1 << k) >= 0:
            want.add(j - (1 << k))
            k += 1
        npred = len(want) - 1                      # predecessors the paper's route reads for block j
        perm = torch.randperm(j, generator=g)[:npred].tolist() if j > 0 else []
        lists.append(sorted(perm) + [j])
    return lists


def mutate_after(w: Workload, q, k, v, seq: int, t: int, seed: int, gain: float = 1.0):
    """Copies of (q, k, v) in which every token of sequence ``seq`` at position > t is
    replaced by fresh finite N(0,1) values (the future-token mutation gate, Section 4.2).
    ``gain`` scales the new Q and K rows: large values make the scores of the mutated rows jump
    from tile to tile by far more than those of the rows that must stay untouched."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    cu = w.cu_seqlens()
    lo, hi = cu[seq] + t + 1, cu[seq + 1]
    q2, k2, v2 = q.clone(), k.clone(), v.clone()
    if hi > lo:
        q2[lo:hi] = (gain * torch.randn((hi - lo, w.hq, w.d), generator=g)).to(torch.bfloat16)
        k2[lo:hi] = (gain * torch.randn((hi - lo, w.hkv, w.d), generator=g)).to(torch.bfloat16)
        v2[lo:hi] = torch.randn((hi - lo, w.hkv, w.d), generator=g).to(torch.bfloat16)
    return q2, k2, v2
