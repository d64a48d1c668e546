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
