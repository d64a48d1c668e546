"""Writes tests/golden/tiny_decode_step.txt: the CPU checker's results for the
tiny fp32 decode configuration (4 layers: standard cache A, sliding ring B of
64 slots, a reader of B, a reader of A; batch 2, 4 query / 2 KV heads x 64;
256 cached tokens, one appended, then attended).

The values come from the checker and the seeded input generators only; the
CUDA library is never called here.  The paper (Section 3) prints no numeric
attention output, so these are not published values: the file freezes what the
checker computed when its pins passed, so that a later change to its
arithmetic, to the cache-indexing rules or to the input generators shows up as
a difference in a text file, and so that the GPU path can be compared with
numbers that no code produces at test time.

Run from the repository root:  python tests/golden/make_golden.py
"""
from __future__ import annotations

import os
import sys

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import mixattn_oracle as mo  # noqa: E402
from synth import configs as cf  # noqa: E402
from synth import inputs as si  # noqa: E402

PATH = os.path.join(HERE, "tiny_decode_step.txt")
CHANNELS = 8      # leading channels of every head that are stored
CHUNK = 100       # the cache is filled in chunks of this many tokens per call


def compute():
    """Returns (state lines, {(layer, seq): [Hq, head_dim] float64 outputs})."""
    wl = cf.tiny_decode()
    dt = torch.float32
    n_pages = wl.batch * (wl.context // wl.page_size + 2)
    ph = mo.PhysicalCache(wl.layout, wl.n_kv_heads, wl.head_dim, wl.batch, n_pages, store_values=True)
    owners = cf.owners_of(wl.layout)
    seqs = list(range(wl.batch))
    # fill: 256 tokens per sequence; rounds of CHUNK tokens for all sequences in one call while
    # every sequence has that many left, then the remainders one sequence per call
    pos = 0
    while pos < wl.context:
        c = min(CHUNK, wl.context - pos)
        groups = [seqs] if c == CHUNK else [[b] for b in seqs]
        for grp in groups:
            for o in owners:
                kv = [si.kv_tokens(wl.seed, o, b, pos, c, wl.n_kv_heads, wl.head_dim, dt) for b in grp]
                K = torch.cat([k for k, _ in kv])
                V = torch.cat([v for _, v in kv])
                ph.append(o, grp, [c] * len(grp), K.numpy(), V.numpy())
        pos += c
    # the step: append position 256 to every owner, then every layer attends
    outs = {}
    for l, (kind, W, owner) in enumerate(wl.layout):
        if owner == l:
            K = torch.cat([si.kv_tokens(wl.seed, l, b, wl.context, 1, wl.n_kv_heads, wl.head_dim, dt)[0] for b in seqs])
            V = torch.cat([si.kv_tokens(wl.seed, l, b, wl.context, 1, wl.n_kv_heads, wl.head_dim, dt)[1] for b in seqs])
            ph.append(l, seqs, None, K.numpy(), V.numpy())
        for b in seqs:
            q = si.q_tokens(wl.seed, l, b, wl.context, 1, wl.n_q_heads, wl.head_dim, dt)[0]
            outs[(l, b)] = np.asarray(ph.decode(l, b, q.double().numpy()), dtype=np.float64)
    state = []
    for b in seqs:
        state.append(f"block_table {b} " + " ".join(str(p) for p in ph.get_block_table(b)))
    for l, (kind, W, owner) in enumerate(wl.layout):
        for b in seqs:
            state.append(f"len {l} {b} {ph.get_len(l, b)}")
            if kind == cf.SLIDING:
                nxt, valid = ph.get_ring_state(l, b)
                state.append(f"ring {l} {b} {nxt} {valid}")
            page, slot = ph.locate(l, b, wl.context)
            state.append(f"locate {l} {b} {wl.context} {page} {slot}")
    state.append(f"free_pages {ph.n_free_pages()}")
    return state, outs


def render() -> str:
    state, outs = compute()
    lines = [
        "# tiny fp32 decode configuration, seed 0: cache state after the step and the first",
        f"# {CHANNELS} channels of every head's output, float64, written by tests/golden/make_golden.py",
        "# from the CPU checker alone (the paper, Section 3, prints no numeric output to cite).",
    ]
    lines += state
    for (l, b), o in sorted(outs.items()):
        for h in range(o.shape[0]):
            lines.append(f"out {l} {b} {h} " + " ".join(f"{x:.17e}" for x in o[h, :CHANNELS]))
    return "\n".join(lines) + "\n"


if __name__ == "__main__":
    with open(PATH, "w") as f:
        f.write(render())
    print("wrote", PATH)
