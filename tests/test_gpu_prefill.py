"""Prompt-attention parity on a B200 against the CPU checker, plus the cache
state a prompt leaves behind (pages, ring contents) and decode after prefill."""
import numpy as np
import pytest
import torch

from oracle import mixattn_oracle as mo
from synth import configs as cf
from synth import inputs as si

from gpu_common import check_close, check_stored_bits, compare_state, load_lib, ref_decode, torch_dt

pytestmark = pytest.mark.gpu


def run_prefill_case(wl: cf.Workload, rows=None, decode_after=True):
    mx, runner = load_lib()
    sess = runner.Session(wl, [0] * wl.batch, headroom_tokens=2)
    ph = mo.PhysicalCache(wl.layout, wl.n_kv_heads, wl.head_dim, wl.batch, sess.n_pages, store_values=False)
    sess.mirror = ph
    S = wl.seq_len
    dt = torch_dt(wl.dtype)
    try:
        for l, (kind, W, owner) in enumerate(wl.layout):
            q, k, v = sess.prefill_inputs(l)
            out = torch.full_like(q, float("nan"))
            sess.prefill_layer(l, q, k, v, out)
            torch.cuda.synchronize()
            got = out.float().cpu().double().numpy().reshape(wl.batch, S, wl.n_q_heads, wl.head_dim)
            for b in range(wl.batch):
                qc = si.q_tokens(wl.seed, l, b, 0, S, wl.n_q_heads, wl.head_dim, dt)
                Kc, Vc = si.kv_tokens(wl.seed, owner, b, 0, S, wl.n_kv_heads, wl.head_dim, dt)
                rs = list(range(S)) if rows is None else [r for r in rows if r < S]
                ref = mo.prefill_attention(qc, Kc, Vc, kind, W, rows=rs)
                check_close(got[b][rs], ref, wl.dtype, f"prefill layer {l} seq {b}")
        assert sess.ctx.get_device_status() == 0
        compare_state(sess.ctx, ph, wl)
        sess.pos[:] = S
        for l, (kind, W, owner) in enumerate(wl.layout):
            lo = 0 if kind == cf.FULL else max(0, S - W)
            for b in range(wl.batch):
                check_stored_bits(sess.ctx, ph, wl, l, b, sorted({lo, S - 1, (lo + S) // 2}))
        if decode_after:
            inputs = sess.step_inputs()
            outs = sess.alloc_outputs()
            sess.decode_step(inputs, outs)
            torch.cuda.synchronize()
            compare_state(sess.ctx, ph, wl)
            got = outs.float().cpu().double().numpy()
            for l in range(len(wl.layout)):
                for b in range(wl.batch):
                    check_close(got[l, b], ref_decode(wl, l, b, S + 1), wl.dtype, f"decode after prefill {l}/{b}")
    finally:
        sess.close()


@pytest.mark.parametrize("S", [1, 31, 32, 33, 200])
def test_prefill_fp32_tiny_layout(S):
    wl = cf.tiny_decode().scaled(seq_len=S, context=0)
    run_prefill_case(wl)


@pytest.mark.parametrize("S,W", [(700, 256), (300, 1024), (129, 128), (1, 16)])
def test_prefill_bf16_small(S, W):
    wl = cf.prefill_chunk().scaled(layout=cf.layout_tiny(W), batch=2, seq_len=S)
    run_prefill_case(wl)


@pytest.mark.parametrize("S,W", [(700, 256), (333, 1024), (129, 128)])
def test_prefill_bf16_head_dim_64(S, W):
    # the tensor-core kernel's 64-channel form: one operand block per tile, 64 accumulator columns
    wl = cf.prefill_chunk().scaled(layout=cf.layout_tiny(W), batch=2, seq_len=S, n_q_heads=12, n_kv_heads=3, head_dim=64)
    run_prefill_case(wl)


def test_prefill_bf16_mid_layout_small():
    wl = cf.prefill_chunk().scaled(layout=cf.layout_mid(256, 6), batch=2, seq_len=600)
    rows = [0, 1, 127, 128, 255, 256, 257, 599] + list(range(300, 340))
    run_prefill_case(wl, rows=rows)


def test_prefill_errors():
    mx, runner = load_lib()
    wl = cf.tiny_decode().scaled(seq_len=8, context=0)
    sess = runner.Session(wl, [0, 0], headroom_tokens=40)
    try:
        q, k, v = sess.prefill_inputs(0)
        out = torch.empty_like(q)
        sess.ctx.prefill(0, [0, 1], [8, 8], q, k, v, out)
        assert sess.ctx.rc_prefill(0, [0], [8], q, k, v, out) == mx.ERR_UNSUPPORTED   # cache not empty
        assert sess.ctx.rc_prefill(0, [0, 0], [8, 8], q, k, v, out) == mx.ERR_INVALID_ARG
        assert sess.ctx.rc_prefill(0, [0], [0], q, k, v, out) == mx.ERR_INVALID_ARG
        assert sess.ctx.rc_prefill(3, [0, 1], [8, 8], q, k, v, out) == 0                 # a reader may re-run
        assert sess.ctx.get_len(3, 0) == 8
        torch.cuda.synchronize()
    finally:
        sess.close()


def _prefill_direct(mx, wl, seq_lens, layer):
    """One prefill call with per-sequence lengths (packed tensors); returns (out, q, k, v) on the CPU."""
    dt = torch_dt(wl.dtype)
    kind, W, owner = wl.layout[layer]
    qs, ks, vs = [], [], []
    for b, S in enumerate(seq_lens):
        qs.append(si.q_tokens(wl.seed, layer, b, 0, S, wl.n_q_heads, wl.head_dim, dt))
        K, V = si.kv_tokens(wl.seed, owner, b, 0, S, wl.n_kv_heads, wl.head_dim, dt)
        ks.append(K)
        vs.append(V)
    return torch.cat(qs), torch.cat(ks), torch.cat(vs)


@pytest.mark.parametrize("hq,hkv,d,dtype", [(8, 8, 128, cf.BF16), (12, 3, 128, cf.BF16), (2, 1, 128, cf.BF16),
                                            (8, 2, 64, cf.BF16), (16, 1, 64, cf.BF16), (6, 3, 128, cf.F32), (6, 3, 64, cf.F32)])
def test_prefill_head_shapes_and_ragged_lengths(hq, hkv, d, dtype):
    # MHA, the paper's 12/3, a single pair, head_dim 64, fp32 (CUDA-core path); sequences of
    # different lengths packed in one call, one of them a single token
    mx, runner = load_lib()
    seq_lens = [333, 129, 1, 128]
    wl = cf.prefill_chunk().scaled(layout=cf.layout_tiny(100), batch=len(seq_lens), seq_len=max(seq_lens),
                                   n_q_heads=hq, n_kv_heads=hkv, head_dim=d, dtype=dtype)
    sess = runner.Session(wl, [0] * wl.batch, headroom_tokens=2)
    ph = mo.PhysicalCache(wl.layout, hkv, d, wl.batch, sess.n_pages, store_values=False)
    try:
        ids = list(range(wl.batch))
        for l, (kind, W, owner) in enumerate(wl.layout):
            q, k, v = _prefill_direct(mx, wl, seq_lens, l)
            qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
            out = torch.full_like(qd, float("nan"))
            sess.ctx.prefill(l, ids, seq_lens, qd, kd, vd, out)
            if owner == l:
                ph.append(l, ids, seq_lens)
            torch.cuda.synchronize()
            got = out.float().cpu().double().numpy()
            row = 0
            for b, S in enumerate(seq_lens):
                ref = mo.prefill_attention(q[row:row + S], k[row:row + S], v[row:row + S], kind, W)
                check_close(got[row:row + S], ref, wl.dtype, f"layer {l} seq {b} len {S}")
                row += S
        assert sess.ctx.get_device_status() == 0
        compare_state(sess.ctx, ph, wl)
        sess.pos[:] = seq_lens
        for b, S in enumerate(seq_lens):
            check_stored_bits(sess.ctx, ph, wl, 1, b, sorted({max(0, S - 100), S - 1}))
            check_stored_bits(sess.ctx, ph, wl, 0, b, sorted({0, S // 2, S - 1}))
    finally:
        sess.close()


@pytest.mark.parametrize("gain", [40.0, 300.0])
def test_prefill_scores_that_outrun_the_exponent_reference(gain):
    # queries scaled so that later tiles hold scores far above the first tile's maximum: the
    # kernel has to move its exponent reference, rescale what it accumulated and recompute
    # the tile; the softmax is close to one-hot and must still match
    mx, runner = load_lib()
    seq_lens = [700, 300]
    wl = cf.prefill_chunk().scaled(layout=cf.layout_tiny(256), batch=len(seq_lens), seq_len=max(seq_lens))
    sess = runner.Session(wl, [0] * wl.batch, headroom_tokens=2)
    try:
        ids = list(range(wl.batch))
        for l in (3, 2):     # readers of the standard and of the sliding cache
            kind, W, owner = wl.layout[l]
            q, k, v = _prefill_direct(mx, wl, seq_lens, l)
            q = (q.float() * gain).to(q.dtype)
            qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
            out = torch.full_like(qd, float("nan"))
            sess.ctx.prefill(l, ids, seq_lens, qd, kd, vd, out)
            torch.cuda.synchronize()
            got = out.float().cpu().double().numpy()
            row = 0
            for b, S in enumerate(seq_lens):
                ref = mo.prefill_attention(q[row:row + S], k[row:row + S], v[row:row + S], kind, W)
                # outputs here are single V rows or mixes of two or three of them, of magnitude up
                # to ~4, not long averages: bf16 rounding of the output (2^-9 relative) and of the
                # few weights that matter (2^-9 each, times |v| <= 5) bound the error
                err = np.abs(got[row:row + S] - ref)
                bound = 1e-2 + 2.0 ** -8 * np.abs(ref) + 2.0 ** -8 * 5.0
                assert (err <= bound).all(), f"gain {gain} layer {l} seq {b}: worst excess {(err - bound).max():.3e}"
                assert err.mean() <= 2e-3
                row += S
        assert sess.ctx.get_device_status() == 0
    finally:
        sess.close()


def test_many_short_prompts_repeated_calls():
    # 64 prompts of 200 tokens: thousands of work items of one or two key tiles, so the warps that
    # write finished tiles fall behind the ones that compute them; every repetition must give the
    # same bits, and those must match the checker (an accumulator read before its last product
    # has landed shows up here)
    mx, runner = load_lib()
    wl = cf.prefill_chunk().scaled(batch=64, seq_len=200)
    sess = runner.Session(wl, [0] * wl.batch)
    dt = torch_dt(wl.dtype)
    S = wl.seq_len
    try:
        for l in (12, 2):        # readers of the standard and of a sliding-window cache: repeatable
            kind, W, owner = wl.layout[l]
            q, k, v = sess.prefill_inputs(l)
            first = None
            for rep in range(12):
                out = torch.full_like(q, float("nan"))
                sess.prefill_layer(l, q, k, v, out)
                torch.cuda.synchronize()
                if first is None:
                    first = out
                else:
                    assert torch.equal(out.view(torch.int16), first.view(torch.int16)), f"layer {l} repetition {rep}"
            got = first.float().cpu().double().numpy().reshape(wl.batch, S, wl.n_q_heads, wl.head_dim)
            for b in (0, 31, 63):
                qc = si.q_tokens(wl.seed, l, b, 0, S, wl.n_q_heads, wl.head_dim, dt)
                Kc, Vc = si.kv_tokens(wl.seed, owner, b, 0, S, wl.n_kv_heads, wl.head_dim, dt)
                rows = [0, 1, 127, 128, 129, 199]
                ref = mo.prefill_attention(qc, Kc, Vc, kind, W, rows=rows)
                check_close(got[b][rows], ref, wl.dtype, f"layer {l} seq {b}")
        assert sess.ctx.get_device_status() == 0
    finally:
        sess.close()


def test_prefill_bf16_error_budget_over_seeds(capsys):
    # The tensor-core prompt kernel against the checker over several seeds, with the error split
    # into the part no bf16 kernel can avoid (rounding the exact result to bf16: |bf16(ref) - ref|)
    # and the kernel's own arithmetic (|got - bf16(ref)|: bf16 weights in the P V product, fp32
    # accumulation order, approximate exponentials).  The tolerances are the usual ones; the two
    # parts are printed (run with -s) so that the margin under the absolute bound is on record.
    mx, runner = load_lib()
    worst = dict(total=0.0, rounding=0.0, arithmetic=0.0)
    for seed in (3, 11, 12, 13, 14, 15):
        wl = cf.prefill_chunk().scaled(layout=cf.layout_tiny(128), batch=2, seq_len=300, seed=seed)
        sess = runner.Session(wl, [0] * wl.batch, headroom_tokens=2)
        dt = torch_dt(wl.dtype)
        S = wl.seq_len
        try:
            for l, (kind, W, owner) in enumerate(wl.layout):
                q, k, v = sess.prefill_inputs(l)
                out = torch.full_like(q, float("nan"))
                sess.prefill_layer(l, q, k, v, out)
                torch.cuda.synchronize()
                got = out.float().cpu().double().numpy().reshape(wl.batch, S, wl.n_q_heads, wl.head_dim)
                for b in range(wl.batch):
                    qc = si.q_tokens(wl.seed, l, b, 0, S, wl.n_q_heads, wl.head_dim, dt)
                    Kc, Vc = si.kv_tokens(wl.seed, owner, b, 0, S, wl.n_kv_heads, wl.head_dim, dt)
                    ref = mo.prefill_attention(qc, Kc, Vc, kind, W)
                    check_close(got[b], ref, wl.dtype, f"seed {seed} layer {l} seq {b}")
                    ref_bf16 = torch.from_numpy(ref).to(torch.bfloat16).double().numpy()
                    worst["total"] = max(worst["total"], float(np.abs(got[b] - ref).max()))
                    worst["rounding"] = max(worst["rounding"], float(np.abs(ref_bf16 - ref).max()))
                    worst["arithmetic"] = max(worst["arithmetic"], float(np.abs(got[b] - ref_bf16).max()))
            assert sess.ctx.get_device_status() == 0
        finally:
            sess.close()
    with capsys.disabled():
        print(f"\nprefill bf16 error budget over 6 seeds: max-abs {worst['total']:.3e} = output rounding "
              f"{worst['rounding']:.3e} + kernel arithmetic {worst['arithmetic']:.3e} (bound 1e-2)")
    # rounding the exact result of magnitude 2..4 to bf16 costs up to 2^-7 = 7.8e-3 by itself
    assert worst["rounding"] <= 2.0 ** -7
