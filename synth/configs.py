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


# ---------------------------------------------------------------------------
# The paper's named variants (Sections 5.1 and 5.2, Appendix A).  The text fixes, per variant, how many standard
# attention caches there are, which layer computes them and who shares them; the figures
# that drew the exact layer indices are not part of the text.  What the text leaves open is
# a parameter here, with defaults that follow the pattern it cites (a standard layer every
# sixth layer, sliding-window layers sharing a ring in groups of two or three).
# ---------------------------------------------------------------------------

def layout_from_roles(n_layers: int, window: int, full_layers, full_owner_of, ring_groups=(3, 2)) -> List[Layer]:
    """Standard layers at `full_layers`, each reading the cache of full_owner_of[layer]
    (itself = it computes its own); every run of sliding layers between them is cut into
    ring-sharing groups of the sizes in `ring_groups`, repeated."""
    full = set(full_layers)
    out: List[Layer] = [None] * n_layers
    group_start, group_left, gi = None, 0, 0
    for l in range(n_layers):
        if l in full:
            out[l] = (FULL, 0, full_owner_of[l])
            group_left = 0           # a standard layer ends the running ring group
            continue
        if group_left == 0:
            group_start, group_left = l, ring_groups[gi % len(ring_groups)]
            gi += 1
        out[l] = (SLIDING, window, group_start)
        group_left -= 1
    return out


def _every(n_layers: int, first: int, step: int):
    return list(range(first, n_layers, step))


def layout_ma(n_layers: int = 24, window: int = 1024, step: int = 6, ring_groups=(3, 2)) -> List[Layer]:
    """MA: one standard cache, computed by the first layer; every other standard layer
    (every `step`-th layer and the last one) reads it."""
    full = sorted(set(_every(n_layers, 0, step) + [n_layers - 1]))
    return layout_from_roles(n_layers, window, full, {l: 0 for l in full}, ring_groups)


def layout_ma_endslide(n_layers: int = 24, window: int = 1024, step: int = 6, ring_groups=(3, 2)) -> List[Layer]:
    """MA-EndSlide: MA with a sliding-window layer last."""
    full = _every(n_layers, 0, step)
    if full[-1] == n_layers - 1:
        full = full[:-1]
    return layout_from_roles(n_layers, window, full, {l: 0 for l in full}, ring_groups)


def layout_ma_offset(n_layers: int = 24, window: int = 1024, offset: int = 2, step: int = 6,
                     ring_groups=(3, 2)) -> List[Layer]:
    """MA-Offset: the first standard layer (which computes the one standard cache) sits
    `offset` layers in, after a few sliding-window layers."""
    full = sorted(set(_every(n_layers, offset, step) + [n_layers - 1]))
    return layout_from_roles(n_layers, window, full, {l: offset for l in full}, ring_groups)


def layout_ma_pairs(n_layers: int = 24, window: int = 1024, reader_distance: int = 6, ring_groups=(3, 2)) -> List[Layer]:
    """MA-Pairs: two standard caches, computed at the first and the thirteenth layer, each
    shared with one more standard layer `reader_distance` layers later."""
    a, b = 0, 12
    own = {a: a, a + reader_distance: a, b: b, min(b + reader_distance, n_layers - 1): b}
    return layout_from_roles(n_layers, window, sorted(own), own, ring_groups)


def layout_slideshare(base: List[Layer]) -> List[Layer]:
    """-SlideShare: more sharing among the sliding-window layers: every run of sliding layers
    between two standard layers shares one ring."""
    out: List[Layer] = []
    run_owner = None
    for l, (kind, w, owner) in enumerate(base):
        if kind == FULL:
            out.append((kind, w, owner))
            run_owner = None
        else:
            if run_owner is None:
                run_owner = l
            out.append((kind, w, run_owner))
    return out


def layout_noshare(n_layers: int = 24, window: int = 1024, n_full: int = 1, offset: int = 0, step: int = 6,
                   ring_groups=(3, 2)) -> List[Layer]:
    """MA-NoShare-k: k standard layers, each with a cache of its own (no standard cache is shared)."""
    full = _every(n_layers, offset, step)[:n_full]
    return layout_from_roles(n_layers, window, full, {l: l for l in full}, ring_groups)


def layout_ma_successive(n_layers: int = 24, window: int = 1024, first: int = 0, gap: int = 12, n_pairs: int = 2,
                         ring_groups=(3, 2)) -> List[Layer]:
    """MA-Successive-k (Appendix A.1): standard caches shared between CONSECUTIVE layers.  Pair p
    sits at layers (first + p * gap, first + p * gap + 1): the first computes a standard cache,
    the next reads it.  The four variants differ in where the pairs sit (`first`) and how far
    apart they are (`gap`); the figure that drew them is not part of the text, so both are
    parameters."""
    own = {}
    for p in range(n_pairs):
        a = first + p * gap
        if a + 1 >= n_layers:
            raise ValueError("pair does not fit the model")
        own[a] = a
        own[a + 1] = a
    return layout_from_roles(n_layers, window, sorted(own), own, ring_groups)


PAPER_VARIANTS = {
    "standard": lambda: layout_all_full(24),
    "sliding_window": lambda: layout_all_sliding(24, 1024),
    "MA": layout_ma,
    "MA-EndSlide": layout_ma_endslide,
    "MA-Offset": layout_ma_offset,
    "MA-Pairs": layout_ma_pairs,
    "MA-Offset-SlideShare": lambda: layout_slideshare(layout_ma_offset()),
    "MA-Pairs-SlideShare": lambda: layout_slideshare(layout_ma_pairs()),
    "MA-NoShare-1": lambda: layout_noshare(n_full=1),
    "MA-NoShare-2": lambda: layout_noshare(n_full=2, offset=2, step=12),
    "MA-NoShare-3": lambda: layout_noshare(n_full=3, offset=2, step=8),
    "MA-Successive-1": lambda: layout_ma_successive(first=0, gap=12),
    "MA-Successive-2": lambda: layout_ma_successive(first=2, gap=12),
    "MA-Successive-3": lambda: layout_ma_successive(first=2, gap=6),
    "MA-Successive-4": lambda: layout_ma_successive(first=6, gap=12),
}


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
