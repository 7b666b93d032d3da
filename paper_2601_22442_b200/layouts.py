"""Flat parameter layouts of the benchmark workloads (host logic only).

The update path sees a stage as a flat vector; only its length matters.  These
helpers give the lengths of Llama-shaped decoder stacks split into contiguous
pipeline stages (Section 2.1: P stages, each a contiguous run of layers).
"""
from __future__ import annotations

from typing import Dict, List, Sequence


def llama_stage_numel(d: int, layers: int, ffn: int, vocab: int, stages: int,
                      tied: bool) -> List[int]:
    """Parameters per stage: per layer 4 d^2 (q, k, v, o) + 3 d ffn (gate, up,
    down) + 2 d (two RMSNorm gains); the first stage adds the vocab x d
    embedding, the last the final norm (d) and, if untied, the vocab x d head."""
    if layers % stages:
        raise ValueError("layers must divide evenly into stages")
    per_layer = 4 * d * d + 3 * d * ffn + 2 * d
    out = [per_layer * (layers // stages)] * stages
    out[0] += vocab * d
    out[-1] += d + (0 if tied else vocab * d)
    return out


def coordinate_shard(numel: Sequence[int], rank: int, world: int, align: int = 1024):
    """The coordinate range of every stage that shard ``rank`` of ``world`` holds.

    Coordinates are independent of one another (Appendix A, remark after Theorem 2)
    and the replica average runs over rows that live together, so a stage can be
    cut into ranges that live on different GPUs with no exchange at all.  Returns
    (shard_numel, coord_base): stage j's shard is [coord_base[j], coord_base[j] +
    shard_numel[j]); the cuts are multiples of ``align`` (itself a multiple of 4,
    which the subset rule needs) and the ranges tile the stage exactly.  A stage
    with fewer than ``world`` aligned pieces cannot be cut that far: ValueError.
    """
    if align % 4 or not (0 <= rank < world):
        raise ValueError("align must be a multiple of 4 and 0 <= rank < world")
    sizes, bases = [], []
    for n in numel:
        pieces = (int(n) + align - 1) // align                 # aligned pieces, the last one ragged
        if pieces < world:
            raise ValueError("a stage of %d coordinates has fewer than %d pieces of %d" % (n, world, align))
        lo = (pieces * rank // world) * align
        hi = min((pieces * (rank + 1) // world) * align, int(n))
        sizes.append(max(hi - lo, 0))
        bases.append(min(lo, int(n)))
    return sizes, bases


# The benchmark configurations (R replicas, stage sizes, delay tau, steps).
def workloads() -> Dict[str, dict]:
    return {
        "toy": dict(R=4, numel=[1 << 20, 1 << 20], tau=1, steps=100),
        "llama125m": dict(R=8, numel=llama_stage_numel(768, 12, 2048, 32000, 4, True),
                          tau=2, steps=50),
        "llama350m": dict(R=8, numel=llama_stage_numel(1024, 24, 2816, 32000, 4, True),
                          tau=4, steps=50),
        # small case for profiler captures: larger than L2, a few GB on the device
        "profile": dict(R=4, numel=[1 << 24, 1 << 24], tau=4, steps=8),
        "profile8": dict(R=8, numel=[1 << 23, 1 << 23], tau=4, steps=8),     # the same bytes, eight replicas
        "llama1b": dict(R=4, numel=llama_stage_numel(2048, 16, 5632, 32000, 8, False),
                        tau=4, steps=20),
    }


DEFAULT_HP = dict(p=0.05, ema_beta=0.9, lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8,
                  weight_decay=0.1)
