"""Drives the library over a synthetic workload: builds a context, fills the
caches with seeded K/V through mixattn_append_kv, and runs decode steps and
prompt passes layer by layer.  Used by the tests, the benchmark and the smoke
check.  Every attention and cache operation happens inside the library; this
module only generates inputs and issues the C-ABI calls.
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional, Sequence

import numpy as np
import torch

from synth import configs as cf
from synth import inputs as si
from . import binding as mx


def torch_dtype(dtype: int):
    return torch.bfloat16 if dtype == cf.BF16 else torch.float32


class Session:
    """One context plus the position bookkeeping of a workload.

    `mirror`, if given, receives the same bookkeeping calls as the library
    (`append(layer, seq_ids, n_new)`), so a checker can follow the cache state.
    """

    def __init__(self, wl: cf.Workload, lengths: Optional[Sequence[int]] = None, device: int = 0,
                 headroom_tokens: int = 0, free_order=None, n_pages: Optional[int] = None,
                 mirror=None, chunk_scratch_tokens: int = 0):
        self.wl = wl
        self.device = device
        self.dev = torch.device(f"cuda:{device}")
        self.dt = torch_dtype(wl.dtype)
        B = wl.batch
        if lengths is None:
            lengths = [wl.context] * B
        self.target = np.asarray(lengths, dtype=np.int64)
        self.pos = np.zeros(B, dtype=np.int64)          # tokens appended so far per sequence
        self.owners = cf.owners_of(wl.layout)
        self.has_full = any(wl.layout[o][0] == cf.FULL for o in self.owners)
        max_len = int(self.target.max()) + headroom_tokens + max(wl.seq_len, 0)
        if n_pages is None:
            n_pages = int(sum(-(-(int(n) + headroom_tokens + max(wl.seq_len, 0)) // wl.page_size)
                              for n in self.target)) if self.has_full else 1
            n_pages = max(n_pages, 1)
        self.n_pages = n_pages
        self.free_order = free_order
        self.mirror = mirror
        self.ctx = mx.Context(wl.layout, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, B,
                              n_pages, max_seq_len=max(max_len, 1), free_order=free_order, device=device,
                              chunk_scratch_tokens=chunk_scratch_tokens)

    def close(self):
        self.ctx.close()

    # ------------------------------------------------------------------
    def _append(self, layer, seq_ids, n_new, K, V, stream=None):
        self.ctx.append_kv(layer, seq_ids, n_new, K, V, stream)
        if self.mirror is not None:
            self.mirror.append(layer, list(seq_ids), None if n_new is None else list(n_new))

    def fill(self, chunk: int = 1024):
        """Appends every sequence's context to every owner, `chunk` tokens per
        sequence per round, so the block tables of the sequences interleave."""
        wl = self.wl
        remaining = self.target - self.pos
        while (remaining > 0).any():
            ids = [b for b in range(wl.batch) if remaining[b] >= chunk]
            if ids:
                groups = [(ids, chunk)]
            else:
                groups = [([b], int(remaining[b])) for b in range(wl.batch) if remaining[b] > 0]
            for seqs, n in groups:
                for o in self.owners:
                    K, V = si.kv_tokens_multi(wl.seed, o, seqs, [self.pos[b] for b in seqs], n,
                                              wl.n_kv_heads, wl.head_dim, self.dt, self.dev)
                    K = K.reshape(-1, wl.n_kv_heads, wl.head_dim)
                    V = V.reshape(-1, wl.n_kv_heads, wl.head_dim)
                    self._append(o, seqs, [n] * len(seqs), K, V)
                for b in seqs:
                    self.pos[b] += n
                    remaining[b] -= n
            torch.cuda.synchronize(self.dev)

    # ------------------------------------------------------------------
    def step_inputs(self, device=None) -> Dict[int, Dict[str, torch.Tensor]]:
        """Q for every layer and the new token's K/V for every owner, for the
        decode step that appends position pos[b] to sequence b."""
        wl = self.wl
        device = self.dev if device is None else device
        out: Dict[int, Dict[str, torch.Tensor]] = {}
        B = wl.batch
        for l in range(len(wl.layout)):
            q = si.q_tokens_multi(wl.seed, l, list(range(B)), [int(p) for p in self.pos], 1, wl.n_q_heads,
                                  wl.head_dim, self.dt, device)[:, 0].contiguous()
            ent = {"q": q}
            if l in self.owners:
                K, V = si.kv_tokens_multi(wl.seed, l, list(range(B)), [int(p) for p in self.pos], 1,
                                          wl.n_kv_heads, wl.head_dim, self.dt, device)
                ent["k"] = K.reshape(B, wl.n_kv_heads, wl.head_dim)
                ent["v"] = V.reshape(B, wl.n_kv_heads, wl.head_dim)
            out[l] = ent
        return out

    def alloc_outputs(self) -> torch.Tensor:
        wl = self.wl
        return torch.empty(len(wl.layout), wl.batch, wl.n_q_heads, wl.head_dim, dtype=self.dt, device=self.dev)

    def decode_step(self, inputs, outs: torch.Tensor, stream=None, advance: bool = True):
        """One decode step of the whole model: per layer, append (owners) then attend."""
        wl = self.wl
        ids = list(range(wl.batch))
        for l in range(len(wl.layout)):
            ent = inputs[l]
            if "k" in ent:
                self._append(l, ids, None, ent["k"], ent["v"], stream)
            self.ctx.decode(l, ids, ent["q"], outs[l], stream)
        if advance:
            self.pos += 1

    # ------------------------------------------------------------------
    def prefill_inputs(self, layer: int, device=None):
        """Packed Q, K, V of the prompts (length wl.seq_len each) for `layer`;
        K/V are the owner's."""
        wl = self.wl
        device = self.dev if device is None else device
        owner = wl.layout[layer][2]
        S = wl.seq_len
        q = si.q_tokens_multi(wl.seed, layer, list(range(wl.batch)), [0] * wl.batch, S, wl.n_q_heads,
                              wl.head_dim, self.dt, device).reshape(-1, wl.n_q_heads, wl.head_dim)
        K, V = si.kv_tokens_multi(wl.seed, owner, list(range(wl.batch)), [0] * wl.batch, S,
                                  wl.n_kv_heads, wl.head_dim, self.dt, device)
        return q, K.reshape(-1, wl.n_kv_heads, wl.head_dim), V.reshape(-1, wl.n_kv_heads, wl.head_dim)

    def prefill_layer(self, layer: int, q, k, v, out, stream=None):
        wl = self.wl
        ids = list(range(wl.batch))
        lens = [wl.seq_len] * wl.batch
        self.ctx.prefill(layer, ids, lens, q, k, v, out, stream)
        if self.mirror is not None and wl.layout[layer][2] == layer:
            self.mirror.append(layer, ids, lens)


def kv_bytes_per_step(wl: cf.Workload, lengths_after: Sequence[int]) -> int:
    """KV bytes one decode step reads: per layer and sequence min(n, window)
    (or n) tokens of 2 * Hkv * D elements; a shared cache counts once per
    reading layer."""
    e = 2 if wl.dtype == cf.BF16 else 4
    per_tok = 2 * wl.n_kv_heads * wl.head_dim * e
    total = 0
    for kind, window, _ in wl.layout:
        for n in lengths_after:
            total += (min(int(n), window) if kind == cf.SLIDING else int(n)) * per_tok
    return total
