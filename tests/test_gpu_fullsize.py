"""The five configurations at full size, in the launch configuration the benchmark
times: cache state compared bit for bit for every sequence, outputs compared on
sampled (layer, sequence, head) triples the CPU checker can compute one by one."""
import numpy as np
import pytest
import torch

from oracle import mixattn_oracle as mo
from synth import configs as cf
from synth import inputs as si

from gpu_common import check_close, check_stored_bits, compare_state, load_lib, torch_dt

pytestmark = pytest.mark.gpu


class HeadHistory:
    """K/V of one (owner, sequence, KV head), regenerated on the CPU and extended on demand."""

    def __init__(self, wl):
        self.wl = wl
        self.cache = {}

    def get(self, owner, seq, g, n):
        wl = self.wl
        key = (owner, seq, g)
        K, V = self.cache.get(key, (None, None))
        have = 0 if K is None else K.shape[0]
        if have < n:
            k2, v2 = si.kv_tokens_head(wl.seed, owner, seq, have, n - have, wl.n_kv_heads, wl.head_dim, g,
                                       torch_dt(wl.dtype))
            k2, v2 = k2.double().numpy(), v2.double().numpy()
            K = k2 if K is None else np.concatenate([K, k2])
            V = v2 if V is None else np.concatenate([V, v2])
            self.cache[key] = (K, V)
        return K[:n], V[:n]


def ref_decode_head(wl, hist, layer, seq, head, n):
    kind, W, owner = wl.layout[layer]
    G = wl.n_q_heads // wl.n_kv_heads
    q = si.q_tokens(wl.seed, layer, seq, n - 1, 1, wl.n_q_heads, wl.head_dim, torch_dt(wl.dtype))[0, head]
    if kind == cf.FULL:
        K, V = hist.get(owner, seq, head // G, n)
    else:   # only the window is needed: regenerate just those tokens
        lo = max(0, n - W)
        K, V = si.kv_tokens_head(wl.seed, owner, seq, lo, n - lo, wl.n_kv_heads, wl.head_dim, head // G,
                                 torch_dt(wl.dtype))
        K, V = K.double().numpy(), V.double().numpy()
    return mo.softmax_attend(q.double().numpy(), K, V, 1.0 / np.sqrt(wl.head_dim))


def run_full_decode(wl, lengths, steps, check_steps, layers, seqs, heads, free_order=None):
    mx, runner = load_lib()
    sess = runner.Session(wl, lengths, headroom_tokens=steps, free_order=free_order)
    ph = mo.PhysicalCache(wl.layout, wl.n_kv_heads, wl.head_dim, wl.batch, sess.n_pages,
                          free_order=free_order, store_values=False)
    sess.mirror = ph
    hist = HeadHistory(wl)
    try:
        sess.fill(1024)
        compare_state(sess.ctx, ph, wl)
        outs = sess.alloc_outputs()
        for step in range(steps):
            inputs = sess.step_inputs()
            sess.decode_step(inputs, outs)
            compare_state(sess.ctx, ph, wl)
            if step in check_steps:
                torch.cuda.synchronize()
                assert sess.ctx.get_device_status() == 0
                got = outs.float().cpu().double().numpy()
                assert np.isfinite(got).all()
                for l in layers:
                    for b in seqs:
                        ref = np.stack([ref_decode_head(wl, hist, l, b, h, int(sess.pos[b])) for h in heads])
                        check_close(got[l, b][heads], ref, wl.dtype, f"step {step} layer {l} seq {b}")
        for l in (layers[0], layers[1]):
            kind, W, _ = wl.layout[l]
            for b in seqs:
                n = int(sess.pos[b])
                lo = 0 if kind == cf.FULL else max(0, n - W)
                check_stored_bits(sess.ctx, ph, wl, l, b, sorted({lo, (lo + n) // 2, n - steps, n - 1}))
    finally:
        sess.close()


def test_mid_decode_full_size():
    wl = cf.mid_decode()
    run_full_decode(wl, [wl.context] * wl.batch, steps=2, check_steps={0, 1},
                    layers=[0, 1, 7, 12, 13, 23], seqs=[0, 31], heads=[0, 5, 31])


@pytest.mark.parametrize("pairs", [False, True])
def test_long_decode_full_size(pairs):
    wl = cf.long_decode(pairs=pairs)
    run_full_decode(wl, [wl.context] * wl.batch, steps=1, check_steps={0},
                    layers=[0, 1, 2, 11, 12, 14, 23], seqs=[7], heads=[3, 28])


def test_mixed_serving_full_size():
    wl = cf.mixed_serving()
    lengths = si.draw_lengths(wl.seed, wl.batch, *wl.context_range).tolist()
    n_pages = sum(-(-(n + wl.n_steps) // wl.page_size) for n in lengths)
    perm = si.page_permutation(wl.seed, n_pages)
    short = int(np.argmin(lengths))
    longest = int(np.argmax(lengths))
    run_full_decode(wl, lengths, steps=wl.n_steps, check_steps={0, 1, 15, 16, 17, 127},
                    layers=[0, 1, 12, 13, 23], seqs=[short, longest], heads=[2, 17], free_order=perm)


def test_mid_decode_full_size_quantised_cache():
    # the mid-decode configuration on a quantised cache (FP8 E4M3 elements), at the size and in the
    # launch configuration bench.py times: stored codes and exponents bit for bit at sampled
    # positions, outputs against the checker's attention over the dequantised history
    mx, runner = load_lib()
    wl = cf.mid_decode()
    sess = runner.Session(wl, [wl.context] * wl.batch, headroom_tokens=2, kv_format=mx.KV_FP8_E4M3)
    ph = mo.PhysicalCache(wl.layout, wl.n_kv_heads, wl.head_dim, wl.batch, sess.n_pages, store_values=False)
    sess.mirror = ph
    G = wl.n_q_heads // wl.n_kv_heads
    dt = torch_dt(wl.dtype)
    try:
        sess.fill(1024)
        outs = sess.alloc_outputs()
        sess.decode_step(sess.step_inputs(), outs)
        torch.cuda.synchronize()
        assert sess.ctx.get_device_status() == 0
        compare_state(sess.ctx, ph, wl)
        n = wl.context + 1
        for l, b, h in ((0, 0, 3), (12, 31, 17), (1, 5, 30), (23, 17, 8)):
            kind, W, owner = wl.layout[l]
            lo = 0 if kind == cf.FULL else n - W
            K, V = si.kv_tokens_head(wl.seed, owner, b, lo, n - lo, wl.n_kv_heads, wl.head_dim, h // G, dt)
            # quantise each head vector as the cache does (one KV head at a time: the rule is per head vector)
            Kq = mo.kv_roundtrip(K.double().numpy()[:, None, :])[:, 0]
            Vq = mo.kv_roundtrip(V.double().numpy()[:, None, :])[:, 0]
            q = si.q_tokens(wl.seed, l, b, n - 1, 1, wl.n_q_heads, wl.head_dim, dt)[0, h].double().numpy()
            ref = mo.softmax_attend(q, Kq, Vq, 1.0 / np.sqrt(wl.head_dim))
            check_close(outs[l, b, h].float().cpu().double().numpy(), ref, wl.dtype, f"layer {l} seq {b} head {h}")
        for l, b, pos in ((0, 7, 0), (0, 7, 20001), (12, 30, n - 1), (1, 2, n - 1024), (13, 9, n - 1)):
            owner = wl.layout[l][2]
            K, V = si.kv_tokens(wl.seed, owner, b, pos, 1, wl.n_kv_heads, wl.head_dim, dt)
            kc, kx, vc, vx = sess.ctx.debug_read_kv_fp8(l, b, pos)
            for got_c, got_x, src in ((kc, kx, K), (vc, vx, V)):
                codes, X = mo.quantize_kv(src)
                assert np.array_equal(got_x, X[0]) and np.array_equal(got_c, codes[0]), (l, b, pos)
    finally:
        sess.close()


def test_prefill_full_size_sampled_rows():
    mx, runner = load_lib()
    wl = cf.prefill_chunk()
    sess = runner.Session(wl, [0] * wl.batch)
    ph = mo.PhysicalCache(wl.layout, wl.n_kv_heads, wl.head_dim, wl.batch, sess.n_pages, store_values=False)
    sess.mirror = ph
    S, W = wl.seq_len, 1024
    G = wl.n_q_heads // wl.n_kv_heads
    hist = HeadHistory(wl)
    rng = np.random.default_rng(wl.seed)
    try:
        for l, (kind, Wl, owner) in enumerate(wl.layout):
            q, k, v = sess.prefill_inputs(l)
            out = torch.empty_like(q)
            sess.prefill_layer(l, q, k, v, out)
            if l not in (0, 1, 5, 12, 13, 23):
                continue
            torch.cuda.synchronize()
            got = out.view(wl.batch, S, wl.n_q_heads, wl.head_dim)
            rows = sorted({0, 1, 127, 128, W - 1, W, W + 1, S - 1} | set(int(x) for x in rng.integers(0, S, 24)))
            for b in (0, wl.batch - 1):
                for h in (1, 30):
                    K, V = hist.get(owner, b, h // G, S)
                    qc = si.q_tokens(wl.seed, l, b, 0, S, wl.n_q_heads, wl.head_dim, torch_dt(wl.dtype))[:, h]
                    qc = qc.double().numpy()
                    ref = np.empty((len(rows), wl.head_dim))
                    for a, i in enumerate(rows):
                        lo, hi = mo.key_range(kind, Wl, i)
                        ref[a] = mo.softmax_attend(qc[i], K[lo:hi], V[lo:hi], 1.0 / np.sqrt(wl.head_dim))
                    g = got[b, rows, h].float().cpu().double().numpy()
                    check_close(g, ref, wl.dtype, f"prefill layer {l} seq {b} head {h}")
        torch.cuda.synchronize()
        assert sess.ctx.get_device_status() == 0
        compare_state(sess.ctx, ph, wl)
        sess.pos[:] = S
        for l in (0, 1, 13):
            kind, Wl, _ = wl.layout[l]
            lo = 0 if kind == cf.FULL else S - Wl
            check_stored_bits(sess.ctx, ph, wl, l, 2, [lo, (lo + S) // 2, S - 1])
    finally:
        sess.close()


def test_prefill_full_size_every_row_of_one_sequence():
    # one standard layer (12) and one sliding-window layer (2) of the prefill configuration,
    # checked on ALL 8192 query rows of one sequence for one head of each of the eight KV
    # groups: every work item of the persistent kernel (64 query tiles per head, up to 64 key
    # tiles per row of tiles) is covered for those heads, not a sample of them
    mx, runner = load_lib()
    wl = cf.prefill_chunk()
    sess = runner.Session(wl, [0] * wl.batch)
    S = wl.seq_len
    G = wl.n_q_heads // wl.n_kv_heads
    hist = HeadHistory(wl)
    b = 1
    heads = (0, 5, 10, 15, 17, 22, 27, 31)   # one head of each of the eight KV groups
    scale = 1.0 / np.sqrt(wl.head_dim)
    try:
        for l in (12, 2):
            kind, Wl, owner = wl.layout[l]
            assert owner != l          # readers: the call stores nothing
            q, k, v = sess.prefill_inputs(l)
            out = torch.full_like(q, float("nan"))
            sess.prefill_layer(l, q, k, v, out)
            torch.cuda.synchronize()
            got = out.view(wl.batch, S, wl.n_q_heads, wl.head_dim)[b].float().cpu().double().numpy()
            qc = si.q_tokens(wl.seed, l, b, 0, S, wl.n_q_heads, wl.head_dim, torch_dt(wl.dtype)).double().numpy()
            for h in heads:
                K, V = hist.get(owner, b, h // G, S)
                ref = np.empty((S, wl.head_dim))
                for i in range(S):
                    lo, hi = mo.key_range(kind, Wl, i)
                    ref[i] = mo.softmax_attend(qc[i, h], K[lo:hi], V[lo:hi], scale)
                check_close(got[:, h], ref, wl.dtype, f"prefill layer {l} seq {b} head {h}, all rows")
        assert sess.ctx.get_device_status() == 0
    finally:
        sess.close()


def test_prefill_served_in_chunks_full_size_sampled_rows():
    # the prefill configuration's prompts (batch 4 x 8192) served in chunks of 2048 behind the cached
    # prefix, in the launch configuration bench.py times; sampled rows of sampled heads per round
    mx, runner = load_lib()
    wl = cf.prefill_chunk().scaled(seq_len=0)
    S, C, W = 8192, 2048, 1024
    sess = runner.Session(wl, [S] * wl.batch, headroom_tokens=1, chunk_scratch_tokens=wl.batch * S)
    ph = mo.PhysicalCache(wl.layout, wl.n_kv_heads, wl.head_dim, wl.batch, sess.n_pages, store_values=False)
    sess.mirror = ph
    G = wl.n_q_heads // wl.n_kv_heads
    hist = HeadHistory(wl)
    rng = np.random.default_rng(wl.seed + 1)
    dt = torch_dt(wl.dtype)
    try:
        for rnd in range(S // C):
            P = rnd * C
            sess.target[:] = P + C
            outs = sess.prefill_in_chunks(C)
            torch.cuda.synchronize()
            rows = sorted({0, 1, 127, 128, C - 1} | set(int(x) for x in rng.integers(0, C, 8)))
            for l in (0, 1, 12, 13, 23):
                kind, Wl, owner = wl.layout[l]
                got = outs[l].view(wl.batch, C, wl.n_q_heads, wl.head_dim)
                for b, h in ((0, 1), (wl.batch - 1, 30)):
                    K, V = hist.get(owner, b, h // G, S)
                    qc = si.q_tokens(wl.seed, l, b, P, C, wl.n_q_heads, wl.head_dim, dt)[:, h].double().numpy()
                    ref = np.empty((len(rows), wl.head_dim))
                    for a, i in enumerate(rows):
                        lo, hi = mo.key_range(kind, Wl, P + i)
                        ref[a] = mo.softmax_attend(qc[i], K[lo:hi], V[lo:hi], 1.0 / np.sqrt(wl.head_dim))
                    g = got[b, rows, h].float().cpu().double().numpy()
                    check_close(g, ref, wl.dtype, f"round {rnd} layer {l} seq {b} head {h}")
        assert sess.ctx.get_device_status() == 0
        compare_state(sess.ctx, ph, wl)
        for l in (0, 1, 13):
            kind, Wl, _ = wl.layout[l]
            lo = 0 if kind == cf.FULL else S - Wl
            check_stored_bits(sess.ctx, ph, wl, l, 2, [lo, (lo + S) // 2, S - 1])
    finally:
        sess.close()
