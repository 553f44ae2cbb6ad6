"""Named synthetic workloads: shapes only, no arithmetic.

The shapes follow two public model families (32 layers, 32/8 heads, head_dim 128;
28 layers, 28/4 heads, head_dim 128) and stand in for reasoning traces of a few
thousand to tens of thousands of tokens.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    q_heads: int
    kv_heads: int
    head_dim: int
    batch: int
    context: int            # tokens already cached when the timed step starts
    frac_compressed: float  # fraction of the layers*kv_heads KV heads that are compressed
    sink: int
    window: int
    seed: int

    @property
    def group(self) -> int:
        return self.q_heads // self.kv_heads

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = {
    # 1 layer, one full and one compressed KV head (the mask is fixed, not drawn)
    "tiny": Workload("tiny", 1, 8, 2, 64, 1, 512, 0.5, 4, 60, 0),
    "llama8b": Workload("llama8b", 32, 32, 8, 128, 16, 8192, 0.20, 16, 112, 1),
    "qwen7b": Workload("qwen7b", 28, 28, 4, 128, 32, 16384, 0.60, 16, 112, 2),
    # long chain-of-thought loop: prompt of 4096 tokens, then 28672 generated steps
    "cot": Workload("cot", 32, 32, 8, 128, 8, 4096, 0.40, 16, 240, 3),
}


def workload_mask(w: Workload) -> "np.ndarray":
    """uint8[layers*kv_heads], 1 = full cache.  The tiny workload fixes its mask (KV head 0 full,
    KV head 1 compressed); every other workload draws it from the seeded global selection."""
    from .generator import head_mask
    if w.name == "tiny":
        return np.array([1, 0] * w.layers, dtype=np.uint8)
    return head_mask(w.seed, w.layers, w.kv_heads, w.frac_compressed)
