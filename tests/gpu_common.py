"""Shared pieces of the GPU parity tests: run a workload through the C ABI and
compare cache state bit for bit and outputs within tolerance with the CPU
checker, on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import mixattn_oracle as mo
from synth import configs as cf
from synth import inputs as si

# tolerances: bf16 I/O with fp32 accumulation; fp32 mode
TOL = {
    cf.BF16: dict(max_abs=1e-2, mean_abs=1e-3, rel_rms=1e-2),
    cf.F32: dict(max_abs=1e-5, mean_abs=1e-6, rel_rms=1e-5),
}


def load_lib():
    from paper_2409_15012_b200 import build as mbuild
    mbuild.build()
    from paper_2409_15012_b200 import binding, runner
    return binding, runner


def check_close(got: np.ndarray, ref: np.ndarray, dtype: int, what: str = ""):
    tol = TOL[dtype]
    err = np.abs(got - ref)
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    assert err.max() <= tol["max_abs"], f"{what}: max-abs {err.max():.3e}"
    assert err.mean() <= tol["mean_abs"], f"{what}: mean-abs {err.mean():.3e}"
    assert rel <= tol["rel_rms"], f"{what}: relative rms {rel:.3e}"
    return float(err.max()), float(rel)


def torch_dt(dtype):
    return torch.bfloat16 if dtype == cf.BF16 else torch.float32


def ref_decode(wl: cf.Workload, layer: int, seq: int, n: int, heads=None) -> np.ndarray:
    """Checker output for the decode of `layer`, sequence `seq`, with n tokens
    in the cache (query at position n-1), from regenerated inputs."""
    kind, window, owner = wl.layout[layer]
    dt = torch_dt(wl.dtype)
    lo = 0 if kind == cf.FULL else max(0, n - window)
    q = si.q_tokens(wl.seed, layer, seq, n - 1, 1, wl.n_q_heads, wl.head_dim, dt)[0]
    G = wl.n_q_heads // wl.n_kv_heads
    if heads is None:
        K, V = si.kv_tokens(wl.seed, owner, seq, lo, n - lo, wl.n_kv_heads, wl.head_dim, dt)
        # the slice [lo, n) is the complete set of keys this layer sees
        return mo.decode_attention(q, K, V, cf.FULL, 0)
    out = np.empty((len(heads), wl.head_dim))
    for r, h in enumerate(heads):
        g = h // G
        K, V = si.kv_tokens_head(wl.seed, owner, seq, lo, n - lo, wl.n_kv_heads, wl.head_dim, g, dt)
        out[r] = mo.softmax_attend(q[h].double().numpy(), K.double().numpy(), V.double().numpy(),
                                   1.0 / np.sqrt(wl.head_dim))
    return out


def compare_state(ctx, ph: mo.PhysicalCache, wl: cf.Workload, seqs=None):
    """Lengths, block tables, ring states and the free count, bit for bit."""
    assert ctx.get_n_free_pages() == ph.n_free_pages()
    for b in (range(wl.batch) if seqs is None else seqs):
        assert ctx.get_block_table(b) == ph.get_block_table(b), f"block table of seq {b}"
        for l, (kind, W, owner) in enumerate(wl.layout):
            assert ctx.get_len(l, b) == ph.get_len(l, b)
            if kind == cf.SLIDING:
                assert ctx.get_ring_state(l, b) == ph.get_ring_state(l, b)


def check_stored_bits(ctx, ph, wl: cf.Workload, layer: int, seq: int, positions):
    """debug_read_kv returns exactly the bits that were appended at `pos`, and
    locate agrees with the checker."""
    dt = torch_dt(wl.dtype)
    owner = wl.layout[layer][2]
    for pos in positions:
        assert ctx.locate(layer, seq, pos) == ph.locate(layer, seq, pos)
        K, V = si.kv_tokens(wl.seed, owner, seq, pos, 1, wl.n_kv_heads, wl.head_dim, dt)
        k, v = ctx.debug_read_kv(layer, seq, pos)
        assert torch.equal(k.view(torch.int16) if dt == torch.bfloat16 else k.view(torch.int32),
                           K[0].view(torch.int16) if dt == torch.bfloat16 else K[0].view(torch.int32))
        assert torch.equal(v.float(), V[0].float())


def run_decode_case(wl: cf.Workload, lengths, steps=1, free_order=None, split_tokens=0, chunk=512,
                    check_layers=None, check_seqs=None, check_heads=None, bits_positions=4):
    """Fills the caches, runs `steps` decode steps, checks state every step and
    outputs every step against the checker.  Returns the outputs of the last step."""
    mx, runner = load_lib()
    sess = runner.Session(wl, lengths, headroom_tokens=steps, free_order=free_order)
    ph = mo.PhysicalCache(wl.layout, wl.n_kv_heads, wl.head_dim, wl.batch, sess.n_pages,
                          free_order=free_order, store_values=False)
    sess.mirror = ph
    try:
        if split_tokens:
            sess.ctx.set_split_tokens(split_tokens)
        sess.fill(chunk)
        compare_state(sess.ctx, ph, wl)
        last = None
        for step in range(steps):
            inputs = sess.step_inputs()
            outs = sess.alloc_outputs()
            outs.fill_(float("nan"))
            sess.decode_step(inputs, outs)
            torch.cuda.synchronize()
            assert sess.ctx.get_device_status() == 0
            compare_state(sess.ctx, ph, wl)
            got = outs.float().cpu().double().numpy()
            for l in (range(len(wl.layout)) if check_layers is None else check_layers):
                for b in (range(wl.batch) if check_seqs is None else check_seqs):
                    n = int(sess.pos[b])
                    ref = ref_decode(wl, l, b, n, check_heads)
                    g = got[l, b] if check_heads is None else got[l, b][list(check_heads)]
                    check_close(g, ref, wl.dtype, f"step {step} layer {l} seq {b} n {n}")
            last = outs
        rng = np.random.default_rng(wl.seed)
        for l in range(len(wl.layout)):
            kind, W, _ = wl.layout[l]
            for b in (range(wl.batch) if check_seqs is None else check_seqs):
                n = int(sess.pos[b])
                lo = 0 if kind == cf.FULL else max(0, n - W)
                cand = {lo, n - 1, (lo + n) // 2} | set(int(x) for x in rng.integers(lo, n, size=bits_positions))
                check_stored_bits(sess.ctx, ph, wl, l, b, sorted(cand))
        return last.clone()
    finally:
        sess.close()
