"""KV-cache capacity of a layer layout: how many tokens fit in a memory budget.

The paper's second headline plot (Section 5.4) is the maximum number of tokens a
model can hold during inference.  With this library's storage rules it is a
closed form of the layout (Section 3): a full-attention OWNER costs
2 * Hkv * D * e bytes per token of context, a sliding-window owner costs a fixed
ring of `window` tokens per sequence, and layers that reuse a cache cost nothing.
The numbers come from the library itself (mixattn_cache_bytes), not from a
re-derivation, so they are what a context would really reserve.
"""
from __future__ import annotations

from typing import Dict, Sequence

from . import binding as mx


def cache_bytes(layout: Sequence, n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: int,
                n_seqs: int, tokens_per_seq: int, kv_format: int = mx.KV_NATIVE) -> int:
    """Bytes of K/V storage for n_seqs sequences of tokens_per_seq tokens each (kv_format:
    native, or the quantised storage of Section 2's "KV Quantization")."""
    n_pages = n_seqs * (-(-tokens_per_seq // 16))
    cfg, keep = mx.make_config(layout, n_q_heads, n_kv_heads, head_dim, dtype, n_seqs, max(n_pages, 1),
                               kv_format=kv_format)
    return mx.cache_bytes(cfg)


def max_sequences(layout: Sequence, n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: int,
                  tokens_per_seq: int, budget_bytes: int, kv_format: int = mx.KV_NATIVE) -> int:
    """Largest batch of sequences of tokens_per_seq tokens whose caches fit in budget_bytes.
    Storage is linear in the number of sequences (pages and rings are per sequence)."""
    per_seq = cache_bytes(layout, n_q_heads, n_kv_heads, head_dim, dtype, 1, tokens_per_seq, kv_format)
    return budget_bytes // per_seq


def capacity_table(layouts: Dict[str, Sequence], n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: int,
                   tokens_per_seq: int, budget_bytes: int, kv_format: int = mx.KV_NATIVE):
    """{name: (bytes per sequence, max sequences, max total tokens)} for each layout."""
    out = {}
    for name, lay in layouts.items():
        per_seq = cache_bytes(lay, n_q_heads, n_kv_heads, head_dim, dtype, 1, tokens_per_seq, kv_format)
        n = max_sequences(lay, n_q_heads, n_kv_heads, head_dim, dtype, tokens_per_seq, budget_bytes, kv_format)
        out[name] = (per_seq, n, n * tokens_per_seq)
    return out
