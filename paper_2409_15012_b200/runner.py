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
                 mirror=None, chunk_scratch_tokens: int = 0, gen_device=None, kv_format: int = mx.KV_NATIVE):
        self.wl = wl
        self.device = device
        self.dev = torch.device(f"cuda:{device}")
        # where the seeded inputs are generated: on the GPU by default (fast for multi-GiB
        # caches); "cpu" generates on the host and copies, so that the only kernels a small run
        # launches are the library's own
        self.gen_dev = self.dev if gen_device is None else torch.device(gen_device)
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
                              chunk_scratch_tokens=chunk_scratch_tokens, kv_format=kv_format)
        self.kv_format = kv_format

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
                                              wl.n_kv_heads, wl.head_dim, self.dt, self.gen_dev)
                    K = K.reshape(-1, wl.n_kv_heads, wl.head_dim).to(self.dev)
                    V = V.reshape(-1, wl.n_kv_heads, wl.head_dim).to(self.dev)
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
        gen = self.gen_dev if device is None else device
        device = self.dev if device is None else device
        out: Dict[int, Dict[str, torch.Tensor]] = {}
        B = wl.batch
        for l in range(len(wl.layout)):
            q = si.q_tokens_multi(wl.seed, l, list(range(B)), [int(p) for p in self.pos], 1, wl.n_q_heads,
                                  wl.head_dim, self.dt, gen)[:, 0].contiguous().to(device)
            ent = {"q": q}
            if l in self.owners:
                K, V = si.kv_tokens_multi(wl.seed, l, list(range(B)), [int(p) for p in self.pos], 1,
                                          wl.n_kv_heads, wl.head_dim, self.dt, gen)
                ent["k"] = K.reshape(B, wl.n_kv_heads, wl.head_dim).to(device)
                ent["v"] = V.reshape(B, wl.n_kv_heads, wl.head_dim).to(device)
            out[l] = ent
        return out

    def alloc_outputs(self) -> torch.Tensor:
        wl = self.wl
        return torch.empty(len(wl.layout), wl.batch, wl.n_q_heads, wl.head_dim, dtype=self.dt, device=self.dev)

    def step_tables(self, inputs, outs: torch.Tensor):
        """Pointer tables of one step's inputs and outputs for mixattn_decode_layers."""
        L = len(self.wl.layout)
        return (self.ctx.pointer_table([inputs[l]["q"] for l in range(L)]),
                self.ctx.pointer_table([inputs[l].get("k") for l in range(L)]),
                self.ctx.pointer_table([inputs[l].get("v") for l in range(L)]),
                self.ctx.pointer_table([outs[l] for l in range(L)]))

    def decode_step(self, inputs, outs: torch.Tensor, stream=None, advance: bool = True, tables=None,
                    layer_range=None):
        """One decode step of the whole model (or of the layers in layer_range): per layer, append
        (owners) then attend, issued as one mixattn_decode_layers call.  `tables` = step_tables(inputs,
        outs) when the caller has built them ahead of time."""
        wl = self.wl
        ids = list(range(wl.batch))
        lo, hi = (0, len(wl.layout)) if layer_range is None else layer_range
        q_tab, k_tab, v_tab, o_tab = self.step_tables(inputs, outs) if tables is None else tables
        self.ctx.decode_layers(lo, hi, ids, q_tab, k_tab, v_tab, o_tab, stream)
        if self.mirror is not None:
            for l in range(lo, hi):
                if wl.layout[l][2] == l:
                    self.mirror.append(l, ids, None)
        if advance:
            self.pos += 1

    # ------------------------------------------------------------------
    def prefill_in_chunks(self, chunk: int, stream=None):
        """Serves what is left of every sequence's prompt (target - pos tokens) in rounds of at
        most `chunk` tokens per sequence: every layer attends the round's chunk behind the cached
        prefix (attend_chunk stores nothing), then every owner appends the round's K/V.  Returns
        the last round's outputs [layers][rows, Hq, D] (sequences back to back)."""
        wl = self.wl
        B, Hq, Hkv, D = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
        outs = None
        while ((self.target - self.pos) > 0).any():
            ids = [b for b in range(B) if self.target[b] > self.pos[b]]
            lens = [int(min(chunk, self.target[b] - self.pos[b])) for b in ids]
            starts = [int(self.pos[b]) for b in ids]
            same = len(set(lens)) == 1

            def q_of(layer):
                if same:
                    return si.q_tokens_multi(wl.seed, layer, ids, starts, lens[0], Hq, D, self.dt,
                                             self.dev).reshape(-1, Hq, D)
                return torch.cat([si.q_tokens(wl.seed, layer, b, p0, n, Hq, D, self.dt, self.dev)
                                  for b, p0, n in zip(ids, starts, lens)])

            def kv_of(owner):
                if same:
                    K, V = si.kv_tokens_multi(wl.seed, owner, ids, starts, lens[0], Hkv, D, self.dt, self.dev)
                    return K.reshape(-1, Hkv, D), V.reshape(-1, Hkv, D)
                kv = [si.kv_tokens(wl.seed, owner, b, p0, n, Hkv, D, self.dt, self.dev)
                      for b, p0, n in zip(ids, starts, lens)]
                return torch.cat([a for a, _ in kv]), torch.cat([c for _, c in kv])

            kv = {o: kv_of(o) for o in self.owners}
            outs = []
            for l, (_, _, owner) in enumerate(wl.layout):
                q = q_of(l)
                out = torch.empty_like(q)
                self.ctx.attend_chunk(l, ids, lens, q, kv[owner][0], kv[owner][1], out, stream)
                outs.append(out)
            for o in self.owners:
                self._append(o, ids, lens, kv[o][0], kv[o][1], stream)
            for b, n in zip(ids, lens):
                self.pos[b] += n
        return outs

    # ------------------------------------------------------------------
    def prefill_inputs(self, layer: int, device=None):
        """Packed Q, K, V of the prompts (length wl.seq_len each) for `layer`;
        K/V are the owner's."""
        wl = self.wl
        gen = self.gen_dev if device is None else device
        device = self.dev if device is None else device
        owner = wl.layout[layer][2]
        S = wl.seq_len
        q = si.q_tokens_multi(wl.seed, layer, list(range(wl.batch)), [0] * wl.batch, S, wl.n_q_heads,
                              wl.head_dim, self.dt, gen).reshape(-1, wl.n_q_heads, wl.head_dim)
        K, V = si.kv_tokens_multi(wl.seed, owner, list(range(wl.batch)), [0] * wl.batch, S,
                                  wl.n_kv_heads, wl.head_dim, self.dt, gen)
        return (q.to(device), K.reshape(-1, wl.n_kv_heads, wl.head_dim).to(device),
                V.reshape(-1, wl.n_kv_heads, wl.head_dim).to(device))

    def prefill_layer(self, layer: int, q, k, v, out, stream=None):
        wl = self.wl
        ids = list(range(wl.batch))
        lens = [wl.seq_len] * wl.batch
        self.ctx.prefill(layer, ids, lens, q, k, v, out, stream)
        if self.mirror is not None and wl.layout[layer][2] == layer:
            self.mirror.append(layer, ids, lens)


def kv_bytes_per_step(wl: cf.Workload, lengths_after: Sequence[int], kv_format: int = mx.KV_NATIVE) -> int:
    """KV bytes one decode step reads: per layer and sequence min(n, window)
    (or n) tokens of 2 * Hkv * D elements (quantised storage: one byte per
    element plus one exponent byte per head vector); a shared cache counts once
    per reading layer."""
    e = 2 if wl.dtype == cf.BF16 else 4
    per_tok = 2 * wl.n_kv_heads * wl.head_dim * e
    if kv_format == mx.KV_FP8_E4M3:
        per_tok = 2 * wl.n_kv_heads * (wl.head_dim + 1)
    n = np.asarray(lengths_after, dtype=np.int64)
    total = 0
    for kind, window, _ in wl.layout:
        total += int((np.minimum(n, window) if kind == cf.SLIDING else n).sum()) * per_tok
    return total


def serve_trace(layout, n_q_heads: int, n_kv_heads: int, head_dim: int, n_requests: int, prompt_len: int,
                gen_len: int, chunk: int, device: int = 0, seed: int = 7, dtype: int = cf.BF16,
                concurrency: int = 0, kv_format: int = mx.KV_NATIVE) -> Dict:
    """Attention-only serving of `n_requests` requests shaped like the paper's benchmark
    (Section 5.4: long prompts, then generated tokens), `concurrency` of them at a time (0 = all
    at once): per wave the prompts in chunks through attend_chunk + append_kv, then `gen_len`
    decode steps, then the sequence slots are reset for the next wave.  `kernel` times are the
    sums of the library's own kernel times (its profile hooks), so input generation is excluded;
    the wall-clock figure beside them includes generating the synthetic inputs on the GPU and
    issuing every call from Python."""
    import time
    conc = n_requests if concurrency <= 0 else min(concurrency, n_requests)
    wl = cf.Workload("serving_trace", list(layout), n_q_heads, n_kv_heads, head_dim, dtype, conc, 0, seed)
    sess = Session(wl, [prompt_len] * conc, device=device, headroom_tokens=gen_len + 1,
                   chunk_scratch_tokens=conc * (prompt_len + chunk), kv_format=kv_format)
    try:
        classes = (mx.K_APPEND, mx.K_DECODE_FULL, mx.K_DECODE_SLIDING, mx.K_COMBINE, mx.K_PREFILL_FULL,
                   mx.K_PREFILL_SLIDING, mx.K_GATHER)
        # prefill_in_chunks hands every reader its owner's K/V tensors, unchanged within a round:
        # the cached keys of a shared cache are copied once per run of layers that read it
        sess.ctx.set_chunk_gather_reuse(True)
        prefill_ms = decode_ms = 0.0
        done, waves = 0, 0
        torch.cuda.synchronize(sess.dev)
        t0 = time.perf_counter()
        while done < n_requests:
            n_wave = min(conc, n_requests - done)
            if waves > 0:
                for b in range(conc):
                    sess.ctx.seq_reset(b)
                sess.pos[:] = 0
            # (a last, smaller wave leaves the other slots empty: their targets are 0)
            sess.target[:] = 0
            sess.target[:n_wave] = prompt_len
            sess.ctx.profile_enable(True)
            sess.prefill_in_chunks(chunk)
            torch.cuda.synchronize(sess.dev)
            prefill_ms += sum(sess.ctx.profile_read(c)[1] for c in classes)
            sess.ctx.profile_enable(True)        # drops the records read so far
            if n_wave == conc:
                outs = sess.alloc_outputs()
                for _ in range(gen_len):
                    sess.decode_step(sess.step_inputs(), outs)
            else:
                decode_partial(sess, n_wave, gen_len)
            torch.cuda.synchronize(sess.dev)
            decode_ms += sum(sess.ctx.profile_read(c)[1] for c in classes)
            sess.ctx.profile_enable(False)
            done += n_wave
            waves += 1
        wall_s = time.perf_counter() - t0
        status = sess.ctx.get_device_status()
        cache = mx.cache_bytes(sess.ctx.cfg)
    finally:
        sess.close()
    tokens = n_requests * (prompt_len + gen_len)
    return {"requests": n_requests, "concurrency": conc, "waves": waves, "prompt_len": prompt_len, "gen_len": gen_len,
            "chunk": chunk, "prefill_kernel_ms": prefill_ms, "decode_kernel_ms": decode_ms,
            "tokens_per_s": tokens / ((prefill_ms + decode_ms) * 1e-3),
            "decode_tokens_per_s": n_requests * gen_len / (decode_ms * 1e-3) if decode_ms > 0 else None,
            "wall_s": wall_s, "wall_tokens_per_s": tokens / wall_s,
            "cache_bytes": cache, "cache_bytes_per_request": cache / conc, "device_status": status}


def decode_partial(sess: Session, n_active: int, steps: int):
    """Decode steps for the first n_active sequence slots only (a last wave that does not fill
    the context)."""
    wl = sess.wl
    ids = list(range(n_active))
    outs = sess.alloc_outputs()
    for _ in range(steps):
        inputs = sess.step_inputs()
        for l in range(len(wl.layout)):
            ent = inputs[l]
            if "k" in ent:
                sess._append(l, ids, None, ent["k"][:n_active], ent["v"][:n_active])
            sess.ctx.decode(l, ids, ent["q"][:n_active], outs[l][:n_active])
        sess.pos[:n_active] += 1
