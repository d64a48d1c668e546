"""Counter-based seeded generator for Q / K / V values, lengths and page orders.

Every value is a pure function of (seed, stream, owner-or-layer, sequence,
token position, head, channel), so any slice of a multi-GiB KV history can be
regenerated anywhere -- on the GPU to fill a cache in chunks, on the CPU for
the few rows a checker wants -- without storing it.

Only integer arithmetic, one int->float conversion and one correctly rounded
fp32 multiply are used, so a CPU tensor and a CUDA tensor built by this code
hold identical bits.  The distribution is Irwin-Hall(8) scaled to zero mean
and unit variance: a close stand-in for N(0,1) (excess kurtosis -0.15,
support +-4.9 sigma) that needs no transcendental function.

The 32-bit mixer is the public-domain "lowbias32" integer hash.
"""
from __future__ import annotations

import numpy as np
import torch

_M32 = 0xFFFFFFFF
_GOLD = 0x9E3779B9
_STREAM_Q = 0x51
_STREAM_KV = 0xC7

# sum of eight uniform 16-bit integers: mean 8*32767.5, variance 8*(2^32-1)/12
_IH_MEAN = 8 * 65535 // 2
_IH_SCALE = float(np.float32(1.0 / np.sqrt(8.0 * (65536.0 ** 2 - 1.0) / 12.0)))


def _mix32_int(x: int) -> int:
    x &= _M32
    x = ((x ^ (x >> 16)) * 0x7FEB352D) & _M32
    x = ((x ^ (x >> 15)) * 0x846CA68B) & _M32
    return x ^ (x >> 16)


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """lowbias32 on an int64 tensor holding values in [0, 2^32)."""
    x = ((x ^ (x >> 16)) * 0x7FEB352D) & _M32
    x = ((x ^ (x >> 15)) * 0x846CA68B) & _M32
    return x ^ (x >> 16)


def stream_key(seed: int, stream: int, a: int, b: int) -> int:
    """32-bit key of one value stream (all arguments are small non-negative ints)."""
    k = _mix32_int(seed * _GOLD + stream)
    k = _mix32_int(k ^ (a * 0x85EBCA6B + 0x1234567))
    k = _mix32_int(k ^ (b * 0xC2B2AE35 + 0x89ABCDE))
    return k


def unit_normal(key, idx: torch.Tensor) -> torch.Tensor:
    """fp32 tensor, one ~N(0,1) value per int64 counter in `idx` (any device).
    `key` is a 32-bit int or an int64 tensor of such keys that broadcasts with idx."""
    x = _mix32((idx & _M32) ^ key)
    x = _mix32(x ^ ((idx >> 32) & _M32))
    acc = torch.zeros_like(idx)
    for r in range(4):
        x = _mix32((x + (_GOLD * (r + 1) & _M32)) & _M32)
        acc = acc + (x & 0xFFFF) + (x >> 16)
    return (acc - _IH_MEAN).to(torch.float32) * _IH_SCALE


def _block(key: int, first: int, shape, dtype, device) -> torch.Tensor:
    n = int(np.prod(shape))
    idx = torch.arange(first, first + n, dtype=torch.int64, device=device)
    return unit_normal(key, idx).to(dtype).reshape(shape)


def kv_tokens(seed, owner, seq, pos0, n, n_kv_heads, head_dim, dtype, device="cpu"):
    """K and V of tokens pos0 .. pos0+n-1 of `seq` in the cache owned by layer `owner`.

    Returns (K, V), each [n, n_kv_heads, head_dim].  The value of a token does
    not depend on how a history is cut into calls.
    """
    key = stream_key(seed, _STREAM_KV, owner, seq)
    per_tok = 2 * n_kv_heads * head_dim
    kv = _block(key, pos0 * per_tok, (n, 2, n_kv_heads, head_dim), dtype, device)
    return kv[:, 0].contiguous(), kv[:, 1].contiguous()


def kv_tokens_multi(seed, owner, seqs, pos0s, n, n_kv_heads, head_dim, dtype, device="cpu"):
    """Same values as kv_tokens for several sequences at once: tokens
    pos0s[i] .. pos0s[i]+n-1 of seqs[i].  Returns (K, V), each
    [len(seqs), n, n_kv_heads, head_dim]."""
    per_tok = 2 * n_kv_heads * head_dim
    keys = torch.tensor([stream_key(seed, _STREAM_KV, owner, int(s)) for s in seqs],
                        dtype=torch.int64, device=device).view(-1, 1)
    first = torch.tensor([int(p) * per_tok for p in pos0s], dtype=torch.int64, device=device).view(-1, 1)
    idx = first + torch.arange(n * per_tok, dtype=torch.int64, device=device).view(1, -1)
    kv = unit_normal(keys, idx).to(dtype).reshape(len(seqs), n, 2, n_kv_heads, head_dim)
    return kv[:, :, 0].contiguous(), kv[:, :, 1].contiguous()


def kv_tokens_head(seed, owner, seq, pos0, n, n_kv_heads, head_dim, g, dtype, device="cpu"):
    """K and V of one KV head `g` only: (K, V), each [n, head_dim]; same values
    as kv_tokens(...)[..][:, g]."""
    key = stream_key(seed, _STREAM_KV, owner, seq)
    pos = torch.arange(pos0, pos0 + n, dtype=torch.int64, device=device).view(n, 1, 1)
    which = torch.arange(2, dtype=torch.int64, device=device).view(1, 2, 1)
    d = torch.arange(head_dim, dtype=torch.int64, device=device).view(1, 1, head_dim)
    idx = ((pos * 2 + which) * n_kv_heads + g) * head_dim + d
    kv = unit_normal(key, idx).to(dtype)
    return kv[:, 0].contiguous(), kv[:, 1].contiguous()


def q_tokens(seed, layer, seq, pos0, n, n_q_heads, head_dim, dtype, device="cpu"):
    """Queries of `layer` for tokens pos0 .. pos0+n-1 of `seq`: [n, n_q_heads, head_dim]."""
    key = stream_key(seed, _STREAM_Q, layer, seq)
    per_tok = n_q_heads * head_dim
    return _block(key, pos0 * per_tok, (n, n_q_heads, head_dim), dtype, device)


def q_tokens_multi(seed, layer, seqs, pos0s, n, n_q_heads, head_dim, dtype, device="cpu"):
    """Same values as q_tokens for several sequences at once:
    [len(seqs), n, n_q_heads, head_dim]."""
    per_tok = n_q_heads * head_dim
    keys = torch.tensor([stream_key(seed, _STREAM_Q, layer, int(s)) for s in seqs],
                        dtype=torch.int64, device=device).view(-1, 1)
    first = torch.tensor([int(p) * per_tok for p in pos0s], dtype=torch.int64, device=device).view(-1, 1)
    idx = first + torch.arange(n * per_tok, dtype=torch.int64, device=device).view(1, -1)
    return unit_normal(keys, idx).to(dtype).reshape(len(seqs), n, n_q_heads, head_dim)


def draw_lengths(seed: int, n: int, lo: int, hi: int) -> np.ndarray:
    """n integers uniform on [lo, hi], both ends included."""
    return np.random.default_rng(seed).integers(lo, hi + 1, size=n).astype(np.int64)


def page_permutation(seed: int, n_pages: int) -> np.ndarray:
    """Seeded permutation of 0..n_pages-1 used as the initial free-page order."""
    return np.random.default_rng(seed + 0x5EED).permutation(n_pages).astype(np.int32)


def sample_pairs(seed: int, n_a: int, n_b: int, count: int):
    """`count` distinct (a, b) pairs with a < n_a, b < n_b, seeded."""
    rng = np.random.default_rng(seed + 0xA11CE)
    total = n_a * n_b
    pick = rng.choice(total, size=min(count, total), replace=False)
    return [(int(p // n_b), int(p % n_b)) for p in pick]
