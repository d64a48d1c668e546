"""Quantised KV storage (FP8 E4M3 elements, shared power-of-two exponent per head vector) on a
B200 against the CPU checker: stored codes and exponents bit for bit, decode and chunk outputs
against the checker's attention over the dequantised cache within the bf16 tolerances."""
import numpy as np
import pytest
import torch

from oracle import mixattn_oracle as mo
from synth import configs as cf
from synth import inputs as si

from gpu_common import check_close, compare_state, load_lib

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def _wl(layout, hq, hkv, batch, seed=5):
    return cf.Workload("fp8_case", layout, hq, hkv, 128, cf.BF16, batch, 0, seed)


def check_stored(ctx, wl, layer, seq, pos):
    owner = wl.layout[layer][2]
    K, V = si.kv_tokens(wl.seed, owner, seq, pos, 1, wl.n_kv_heads, wl.head_dim, BF)
    kc, kx, vc, vx = ctx.debug_read_kv_fp8(layer, seq, pos)
    for got_c, got_x, src in ((kc, kx, K), (vc, vx, V)):
        codes, X = mo.quantize_kv(src)
        assert np.array_equal(got_x, X[0]), f"exponents at layer {layer} seq {seq} pos {pos}"
        assert np.array_equal(got_c, codes[0]), f"codes at layer {layer} seq {seq} pos {pos}"
    k, v = ctx.debug_read_kv(layer, seq, pos)          # dequantised, exact in bf16
    assert np.array_equal(k.double().numpy(), mo.kv_roundtrip(K)[0])
    assert np.array_equal(v.double().numpy(), mo.kv_roundtrip(V)[0])


def ref_decode_q(wl, layer, seq, n):
    kind, W, owner = wl.layout[layer]
    lo = 0 if kind == cf.FULL else max(0, n - W)
    q = si.q_tokens(wl.seed, layer, seq, n - 1, 1, wl.n_q_heads, wl.head_dim, BF)[0]
    K, V = si.kv_tokens(wl.seed, owner, seq, lo, n - lo, wl.n_kv_heads, wl.head_dim, BF)
    exact = mo.decode_attention(q, K, V, cf.FULL, 0)
    return mo.decode_attention(q, mo.kv_roundtrip(K), mo.kv_roundtrip(V), cf.FULL, 0), exact


@pytest.mark.parametrize("hq,hkv,lengths,split", [
    (32, 8, [700, 64, 1, 2100], 0),        # few (sequence, head) pairs of mixed length: single-wave splits
    (12, 3, [5000, 300], 0),               # the paper's heads; at most one item per two SMs: cluster pairs
    (8, 8, [40, 1500, 17], 256),           # one query head per KV head; forced short splits + combine
    (16, 2, [900, 2500, 129], 512),        # eight query heads per KV head
])
def test_fp8_decode_steps_state_bits_and_outputs(hq, hkv, lengths, split):
    mx, runner = load_lib()
    wl = _wl(cf.layout_tiny(512), hq, hkv, len(lengths))
    steps = 3
    sess = runner.Session(wl, lengths, headroom_tokens=steps, kv_format=mx.KV_FP8_E4M3)
    ph = mo.PhysicalCache(wl.layout, hkv, 128, wl.batch, sess.n_pages, store_values=False)
    sess.mirror = ph
    worst_q = 0.0
    try:
        if split:
            sess.ctx.set_split_tokens(split)
        sess.fill(333)
        compare_state(sess.ctx, ph, wl)
        for step in range(steps):
            inputs = sess.step_inputs()
            outs = sess.alloc_outputs()
            outs.fill_(float("nan"))
            sess.decode_step(inputs, outs)
            torch.cuda.synchronize()
            assert sess.ctx.get_device_status() == 0
            compare_state(sess.ctx, ph, wl)
            got = outs.float().cpu().double().numpy()
            for l in range(len(wl.layout)):
                for b in range(wl.batch):
                    ref, exact = ref_decode_q(wl, l, b, int(sess.pos[b]))
                    check_close(got[l, b], ref, wl.dtype, f"step {step} layer {l} seq {b}")
                    worst_q = max(worst_q, float(np.abs(ref - exact).max()))
        for l, (kind, W, _) in enumerate(wl.layout):
            for b in range(wl.batch):
                n = int(sess.pos[b])
                lo = 0 if kind == cf.FULL else max(0, n - W)
                for pos in sorted({lo, n - 1, (lo + n) // 2}):
                    check_stored(sess.ctx, wl, l, b, pos)
        print(f"\nfp8 cache: the quantisation itself moves the outputs by up to {worst_q:.3e} (checker, informative)")
    finally:
        sess.close()


def test_fp8_special_rows_are_stored_as_the_rule_says():
    # rows built to hit the corners of the format: zero vector, a power-of-two maximum, a maximum
    # that saturates (500 -> 448), negative zero, values that underflow to zero, a huge and a tiny row
    mx, runner = load_lib()
    wl = _wl(cf.layout_tiny(64), 4, 2, 1)
    sess = runner.Session(wl, [0], headroom_tokens=40, kv_format=mx.KV_FP8_E4M3)
    try:
        rng = np.random.default_rng(9)
        rows = []
        base = torch.from_numpy(rng.standard_normal((2, 128))).to(BF)
        for scale in (0.0, 1.0, 2.0 ** -20, 2.0 ** 30, 2.0 ** -100, 2.0 ** 100):
            rows.append(base * scale)
        r = base.clone(); r[:, 3] = 8.0; r[:, 5] = -8.0; r.clamp_(-8.0, 8.0); rows.append(r)         # amax = 2^3 exactly
        r = (base * 0.01).clone(); r[:, 7] = 500.0; rows.append(r)                                      # saturates
        r = (base * 0.0).clone(); r[:, 0] = 1.0; r[:, 1] = -0.0; r[:, 2] = 2.0 ** -18; r[:, 4] = -(2.0 ** -19)
        r[:, 6] = 3 * 2.0 ** -18; rows.append(r)                                                        # ties and underflow
        K = torch.stack(rows).to(BF)                  # [n, Hkv, D]
        V = torch.flip(K, dims=[0]).contiguous()
        n = K.shape[0]
        for layer in (0, 1):
            sess.ctx.append_kv(layer, [0], [n], K.cuda(), V.cuda())
        torch.cuda.synchronize()
        for layer in (0, 1):
            for pos in range(n):
                kc, kx, vc, vx = sess.ctx.debug_read_kv_fp8(layer, 0, pos)
                for got_c, got_x, src in ((kc, kx, K[pos:pos + 1]), (vc, vx, V[pos:pos + 1])):
                    codes, X = mo.quantize_kv(src)
                    assert np.array_equal(got_x, X[0]), (layer, pos, got_x, X[0])
                    assert np.array_equal(got_c, codes[0]), (layer, pos)
    finally:
        sess.close()


def test_fp8_chunks_read_the_cache_dequantised_and_decode_follows():
    mx, runner = load_lib()
    wl = _wl(cf.layout_tiny(256), 12, 3, 2)
    schedule = [[300, 130, 1], [50, 400, 64]]
    totals = [sum(s) for s in schedule]
    sess = runner.Session(wl, totals, headroom_tokens=2, chunk_scratch_tokens=1200, kv_format=mx.KV_FP8_E4M3)
    pos = [0, 0]
    try:
        for rnd in range(3):
            ids = [0, 1]
            lens = [schedule[b][rnd] for b in ids]
            for l, (kind, W, owner) in enumerate(wl.layout):
                q = torch.cat([si.q_tokens(wl.seed, l, b, pos[b], n, wl.n_q_heads, 128, BF) for b, n in zip(ids, lens)])
                kv = [si.kv_tokens(wl.seed, owner, b, pos[b], n, wl.n_kv_heads, 128, BF) for b, n in zip(ids, lens)]
                k, v = torch.cat([a for a, _ in kv]), torch.cat([c for _, c in kv])
                out = torch.full_like(q, float("nan"), device="cuda")
                sess.ctx.attend_chunk(l, ids, lens, q.cuda(), k.cuda(), v.cuda(), out)
                torch.cuda.synchronize()
                got = out.float().cpu().double().numpy()
                row = 0
                for b, n in zip(ids, lens):
                    # the cached part reads back quantised, the chunk's own rows are as given
                    Kp, Vp = si.kv_tokens(wl.seed, owner, b, 0, pos[b], wl.n_kv_heads, 128, BF)
                    Kh = np.concatenate([mo.kv_roundtrip(Kp), kv[ids.index(b)][0].double().numpy()])
                    Vh = np.concatenate([mo.kv_roundtrip(Vp), kv[ids.index(b)][1].double().numpy()])
                    ref = mo.prefill_attention(q[row:row + n], Kh, Vh, kind, W, prefix_len=pos[b])
                    check_close(got[row:row + n], ref, wl.dtype, f"round {rnd} layer {l} seq {b}")
                    row += n
            for o in cf.owners_of(wl.layout):
                kv = [si.kv_tokens(wl.seed, o, b, pos[b], n, wl.n_kv_heads, 128, BF) for b, n in zip(ids, lens)]
                sess.ctx.append_kv(o, ids, lens, torch.cat([a for a, _ in kv]).cuda(), torch.cat([c for _, c in kv]).cuda())
            for b, n in zip(ids, lens):
                pos[b] += n
        assert sess.ctx.get_device_status() == 0
        sess.pos[:] = pos
        outs = sess.alloc_outputs()
        sess.decode_step(sess.step_inputs(), outs)
        torch.cuda.synchronize()
        got = outs.float().cpu().double().numpy()
        for l in range(len(wl.layout)):
            for b in range(wl.batch):
                check_close(got[l, b], ref_decode_q(wl, l, b, pos[b] + 1)[0], wl.dtype, f"decode after chunks {l}/{b}")
    finally:
        sess.close()


def test_fp8_prompt_call_stores_quantised_and_rope_append_quantises_the_rotated_keys():
    mx, runner = load_lib()
    wl = _wl(cf.layout_tiny(128), 8, 2, 2).scaled(seq_len=200)
    sess = runner.Session(wl, [0, 0], headroom_tokens=8, kv_format=mx.KV_FP8_E4M3)
    try:
        # prompt call on the owners: attention over the K/V given (unquantised), store quantised
        for l in (0, 1):
            kind, W, owner = wl.layout[l]
            q, k, v = sess.prefill_inputs(l)
            out = torch.full_like(q, float("nan"))
            sess.prefill_layer(l, q, k, v, out)
            torch.cuda.synchronize()
            got = out.float().cpu().double().numpy().reshape(2, 200, wl.n_q_heads, 128)
            for b in range(2):
                qc = si.q_tokens(wl.seed, l, b, 0, 200, wl.n_q_heads, 128, BF)
                Kc, Vc = si.kv_tokens(wl.seed, owner, b, 0, 200, wl.n_kv_heads, 128, BF)
                check_close(got[b], mo.prefill_attention(qc, Kc, Vc, kind, W), wl.dtype, f"prompt layer {l} seq {b}")
            for b in range(2):
                for pos in ((0, 100, 199) if kind == cf.FULL else (72, 150, 199)):
                    check_stored(sess.ctx, wl, l, b, pos)
        # rotary append: the stored row is the quantised form of the rotated key rounded to bf16
        theta = 500000.0
        K = si.kv_tokens(wl.seed, 0, 0, 200, 3, wl.n_kv_heads, 128, BF)[0]
        V = si.kv_tokens(wl.seed, 0, 0, 200, 3, wl.n_kv_heads, 128, BF)[1]
        sess.ctx.append_kv_rope(0, [0], [3], K.cuda(), V.cuda(), theta)
        torch.cuda.synchronize()
        rot = mo.rope_rotate(K, [200, 201, 202], theta)
        for i in range(3):
            kc, kx, vc, vx = sess.ctx.debug_read_kv_fp8(0, 0, 200 + i)
            # the rotation runs in fp32 on the GPU: a rotated value may round to the neighbouring
            # bf16 number, which can move a code by one step; exponents and values must agree with
            # the checker's quantisation of one of the two
            codes, X = mo.quantize_kv(torch.from_numpy(rot[i:i + 1]).to(BF))
            assert np.array_equal(kx, X[0])
            d = np.abs(mo.dequantize_kv(kc[None], kx[None]) - mo.dequantize_kv(codes, X))
            step = np.exp2(X[0].astype(np.float64))[:, None] * 32.0      # largest grid step of the row
            assert (d <= step[None]).all() and (kc == codes[0]).mean() > 0.97
            cv, Xv = mo.quantize_kv(V[i:i + 1])
            assert np.array_equal(vc, cv[0]) and np.array_equal(vx, Xv[0])
    finally:
        sess.close()


def test_fp8_mid_layout_decode_sampled():
    # the 24-layer layout at a few thousand tokens, ragged: the standard launch configuration
    # (8 consumer warps, splits of 4096 keys, combine) and the two-CTA-per-SM one on the rings
    mx, runner = load_lib()
    wl = cf.mid_decode().scaled(batch=24, context=0, name="fp8_mid", seed=6)
    lengths = [int(x) for x in np.random.default_rng(6).integers(1500, 9000, size=wl.batch)]
    sess = runner.Session(wl, lengths, headroom_tokens=2, kv_format=mx.KV_FP8_E4M3)
    try:
        sess.fill(1024)
        outs = sess.alloc_outputs()
        sess.decode_step(sess.step_inputs(), outs)
        torch.cuda.synchronize()
        assert sess.ctx.get_device_status() == 0
        got = outs.float().cpu().double().numpy()
        for l in (0, 1, 7, 12, 13, 23):
            for b in (0, 11, 23):
                check_close(got[l, b], ref_decode_q(wl, l, b, int(sess.pos[b]))[0], wl.dtype, f"layer {l} seq {b}")
    finally:
        sess.close()
