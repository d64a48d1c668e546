"""Layer layouts and the five synthetic workloads (plain data, no arithmetic).

A layout is a list of (kind, window, kv_owner_layer) per layer, following the
paper's Section 3: each layer is a standard or a sliding-window attention layer
and either computes its own KV cache or reuses the cache of an earlier layer.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Tuple

FULL = 0
SLIDING = 1
F32 = 0
BF16 = 1

Layer = Tuple[int, int, int]  # (kind, window, kv_owner_layer)


def layout_tiny(window: int = 64) -> List[Layer]:
    """4 layers: full owner A, sliding owner B, sliding reader of B, full reader of A."""
    return [(FULL, 0, 0), (SLIDING, window, 1), (SLIDING, window, 1), (FULL, 0, 0)]


def layout_mid(window: int = 1024, n_layers: int = 24) -> List[Layer]:
    """One full cache (layer 0, reused by the middle layer) and two shared rings.

    Layer 0 full owner; layers 1..h-1 share the ring of layer 1; layer h reads
    layer 0's cache; layers h+1..L-1 share the ring of layer h+1 (h = L/2).
    """
    h = n_layers // 2
    out: List[Layer] = []
    for l in range(n_layers):
        if l == 0 or l == h:
            out.append((FULL, 0, 0))
        elif l < h:
            out.append((SLIDING, window, 1))
        else:
            out.append((SLIDING, window, h + 1))
    return out


def layout_pairs(window: int = 1024, n_layers: int = 24) -> List[Layer]:
    """Like layout_mid, but sliding layers share in pairs: an odd sliding layer
    owns a ring and the next layer, when it is a sliding layer too, reads it."""
    h = n_layers // 2
    out: List[Layer] = []
    for l in range(n_layers):
        if l == 0 or l == h:
            out.append((FULL, 0, 0))
        elif l % 2 == 1:
            out.append((SLIDING, window, l))
        else:
            out.append((SLIDING, window, l - 1))
    return out


def layout_all_full(n_layers: int) -> List[Layer]:
    return [(FULL, 0, l) for l in range(n_layers)]


def layout_all_sliding(n_layers: int, window: int) -> List[Layer]:
    return [(SLIDING, window, l) for l in range(n_layers)]


def owners_of(layout: List[Layer]) -> List[int]:
    return [l for l, (_, _, o) in enumerate(layout) if o == l]


@dataclass(frozen=True)
class Workload:
    name: str
    layout: List[Layer]
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: int
    batch: int
    context: int              # tokens cached per sequence before the step (fixed-length workloads)
    seed: int
    page_size: int = 16
    seq_len: int = 0          # prefill length (prefill workloads)
    context_range: Tuple[int, int] = (0, 0)   # ragged workloads: inclusive range of lengths
    n_steps: int = 1
    permute_pages: bool = False
    notes: str = ""

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


def tiny_decode() -> Workload:
    return Workload("tiny_decode_fp32", layout_tiny(64), 4, 2, 64, F32, 2, 256, seed=0)


def mid_decode() -> Workload:
    return Workload("mid_decode_bf16", layout_mid(1024), 32, 8, 128, BF16, 32, 32768, seed=1)


def long_decode(pairs: bool = False) -> Workload:
    lay = layout_pairs(1024) if pairs else layout_mid(1024)
    return Workload("long_decode_bf16" + ("_pairs" if pairs else ""), lay, 32, 8, 128, BF16, 8,
                    131072, seed=2)


def prefill_chunk() -> Workload:
    return Workload("prefill_bf16", layout_mid(1024), 32, 8, 128, BF16, 4, 0, seed=3, seq_len=8192)


def mixed_serving() -> Workload:
    return Workload("mixed_serving_bf16", layout_mid(1024), 32, 8, 128, BF16, 64, 0, seed=4,
                    context_range=(1024, 65536), n_steps=128, permute_pages=True)


ALL = {
    "tiny_decode": tiny_decode,
    "mid_decode": mid_decode,
    "long_decode": long_decode,
    "prefill_chunk": prefill_chunk,
    "mixed_serving": mixed_serving,
}
