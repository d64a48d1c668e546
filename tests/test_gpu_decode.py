"""Decode parity on a B200: the library through its C ABI against the CPU checker,
element by element at small sizes (several tiles, ragged tails), with the cache
state compared bit for bit."""
import numpy as np
import pytest
import torch

from synth import configs as cf
from synth import inputs as si

from gpu_common import load_lib, run_decode_case

pytestmark = pytest.mark.gpu


def test_tiny_decode_fp32_config():
    # the tiny configuration as specified: 256 cached tokens, one appended, fp32, tolerance 1e-5
    wl = cf.tiny_decode()
    run_decode_case(wl, [wl.context] * wl.batch, steps=2, chunk=100)


@pytest.mark.parametrize("ctx_len", [0, 1, 15, 16, 63, 64, 65, 1000])
def test_fp32_lengths_around_page_and_window_edges(ctx_len):
    wl = cf.tiny_decode().scaled(context=ctx_len)
    run_decode_case(wl, [ctx_len, max(0, ctx_len - 3)], steps=2, chunk=37)


def test_mid_layout_bf16_small():
    # 24 layers, 32/8 heads, D 128, W 1024 with wrapped rings, ragged tails, several splits
    wl = cf.mid_decode().scaled(batch=3, context=2500)
    run_decode_case(wl, [2500, 1023, 1024 + 333], steps=2, chunk=300)


def test_pairs_layout_bf16_small():
    wl = cf.long_decode(pairs=True).scaled(batch=2, context=3000)
    run_decode_case(wl, [3000, 2049], steps=1, chunk=1000)


@pytest.mark.parametrize("n", [1, 2, 15, 16, 17, 63, 64, 65, 255, 256, 257, 1023, 1024, 1025])
def test_bf16_context_lengths(n):
    wl = cf.mid_decode().scaled(layout=cf.layout_tiny(256), batch=2, context=n)
    run_decode_case(wl, [n - 1, max(0, n - 2)], steps=1, chunk=200)


@pytest.mark.parametrize("hq,hkv,d", [(8, 8, 128), (16, 2, 128), (16, 1, 64), (8, 2, 64), (12, 3, 128),
                                      (64, 2, 128), (40, 2, 64)])
def test_bf16_head_shapes(hq, hkv, d):
    # MHA, groups of 8 / 16, the paper's 12/3, groups of 32 and 20 (two passes of 16 rows)
    wl = cf.mid_decode().scaled(layout=cf.layout_tiny(128), batch=2, context=700,
                                n_q_heads=hq, n_kv_heads=hkv, head_dim=d)
    run_decode_case(wl, [700, 150], steps=1, chunk=256)


@pytest.mark.parametrize("hq,hkv,d", [(8, 8, 128), (6, 1, 64), (40, 2, 128)])
def test_fp32_head_shapes(hq, hkv, d):
    wl = cf.tiny_decode().scaled(batch=2, context=300, n_q_heads=hq, n_kv_heads=hkv, head_dim=d)
    run_decode_case(wl, [300, 70], steps=1, chunk=128)


def test_results_independent_of_split_count():
    wl = cf.mid_decode().scaled(layout=cf.layout_tiny(512), batch=2, context=3000)
    outs = [run_decode_case(wl, [3000, 1700], split_tokens=s, chunk=1000).float() for s in (0, 16, 64, 500, 100000)]
    for o in outs[1:]:
        assert (o - outs[0]).abs().max().item() <= 4e-3      # bf16 output rounding only
    wl32 = cf.tiny_decode().scaled(context=900)
    outs = [run_decode_case(wl32, [900, 500], split_tokens=s, chunk=1000) for s in (0, 16, 100000)]
    for o in outs[1:]:
        rel = ((o - outs[0]).norm() / outs[0].norm()).item()
        assert rel <= 1e-6


def test_page_permutation_leaves_outputs_bit_identical():
    wl = cf.mid_decode().scaled(layout=cf.layout_tiny(256), batch=3, context=1500)
    lengths = [1500, 800, 47]
    a = run_decode_case(wl, lengths, steps=2, chunk=128)
    n_pages = sum(-(-(n + 2) // 16) for n in lengths)
    perm = si.page_permutation(wl.seed, n_pages)
    b = run_decode_case(wl, lengths, steps=2, chunk=128, free_order=perm)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_ragged_serving_small():
    # scaled-down mixed serving: ragged lengths, permuted pages, rings at arbitrary
    # offsets, 20 steps with appends crossing page boundaries
    wl = cf.mixed_serving().scaled(layout=cf.layout_mid(256), batch=6, n_steps=20)
    lengths = si.draw_lengths(wl.seed, wl.batch, 64, 3000).tolist()
    lengths[0] = 256
    lengths[1] = 15
    n_pages = sum(-(-(n + 20) // 16) for n in lengths)
    run_decode_case(wl, lengths, steps=20, chunk=100, free_order=si.page_permutation(wl.seed, n_pages),
                    check_layers=[0, 1, 7, 12, 13, 23])


def test_large_batch_is_chunked_over_launches():
    # more sequences than one launch carries metadata for
    wl = cf.mid_decode().scaled(layout=cf.layout_tiny(64), batch=150, context=90, n_q_heads=8, n_kv_heads=2)
    run_decode_case(wl, [90 + (b % 7) for b in range(150)], steps=1, chunk=64,
                    check_seqs=[0, 1, 127, 128, 149], bits_positions=1)


def test_decode_errors_write_nothing():
    from gpu_common import load_lib
    mx, runner = load_lib()
    wl = cf.tiny_decode()
    sess = runner.Session(wl, [5, 0], headroom_tokens=1)
    try:
        sess.fill()
        q = torch.zeros(2, wl.n_q_heads, wl.head_dim, device="cuda")
        out = torch.full_like(q, 7.0)
        assert sess.ctx.rc_decode(0, [0, 1], q, out) == mx.ERR_EMPTY_CONTEXT
        assert sess.ctx.rc_decode(0, [0, 2], q, out) == mx.ERR_BAD_SEQ
        assert sess.ctx.rc_append_kv(3, [0], None, q, q) == mx.ERR_NOT_OWNER
        torch.cuda.synchronize()
        assert (out == 7.0).all()
        assert sess.ctx.get_launch_count() > 0
    finally:
        sess.close()


def test_repeated_calls_are_bit_identical_and_profile_hooks_count():
    # the same decode / prefill call twice gives the same bits (no order-dependent reduction
    # across CTAs), and the per-kernel event hooks see every launch
    from gpu_common import load_lib
    mx, runner = load_lib()
    wl = cf.mid_decode().scaled(batch=5, context=9000)
    sess = runner.Session(wl, [9000, 4097, 1024, 300, 17], headroom_tokens=2)
    try:
        sess.fill(1500)
        inputs = sess.step_inputs()
        outs = sess.alloc_outputs()
        sess.decode_step(inputs, outs)
        ids = list(range(wl.batch))
        sess.ctx.profile_enable(True)
        for l in (0, 1, 5, 12, 23):
            a = torch.empty_like(outs[l])
            b = torch.empty_like(outs[l])
            sess.ctx.decode(l, ids, inputs[l]["q"], a)
            sess.ctx.decode(l, ids, inputs[l]["q"], b)
            torch.cuda.synchronize()
            assert torch.equal(a.view(torch.int16), b.view(torch.int16))
            assert torch.equal(a.view(torch.int16), outs[l].view(torch.int16))
        n_full, ms_full = sess.ctx.profile_read(mx.K_DECODE_FULL)
        n_slide, ms_slide = sess.ctx.profile_read(mx.K_DECODE_SLIDING)
        n_comb, _ = sess.ctx.profile_read(mx.K_COMBINE)
        assert (n_full, n_slide) == (4, 6) and ms_full > 0 and ms_slide > 0 and n_comb == 4
        sess.ctx.profile_enable(False)
        assert sess.ctx.get_device_status() == 0
    finally:
        sess.close()
    wl = cf.prefill_chunk().scaled(layout=cf.layout_tiny(256), batch=2, seq_len=700)
    sess = runner.Session(wl, [0, 0])
    try:
        for l in (2, 3):      # readers: repeatable, store nothing
            q, k, v = sess.prefill_inputs(l)
            a, b = torch.empty_like(q), torch.empty_like(q)
            sess.prefill_layer(l, q, k, v, a)
            sess.prefill_layer(l, q, k, v, b)
            torch.cuda.synchronize()
            assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    finally:
        sess.close()


def test_bf16_few_items_short_and_long_sequences_together():
    # a launch of few items gives every item two CTAs that halve its keys: a sequence of one
    # stage or less leaves the second CTA without keys, 65 keys give it a single one
    wl = cf.mid_decode().scaled(layout=cf.layout_tiny(512), batch=4, context=1000, n_q_heads=16, n_kv_heads=4)
    run_decode_case(wl, [1000, 4, 63, 64], steps=2, chunk=250)


def test_decode_layers_is_the_per_layer_calls():
    # one mixattn_decode_layers call over all layers, and over two ranges, against the individual
    # append_kv / decode calls: same cache state, same bits
    mx, runner = load_lib()
    wl = cf.mid_decode().scaled(layout=cf.layout_mid(256, 6), batch=3, context=0)
    lengths = [700, 40, 2100]
    outs_by_mode = []
    for mode in ("calls", "one", "ranges"):
        sess = runner.Session(wl, lengths, headroom_tokens=3)
        try:
            sess.fill(512)
            ids = list(range(wl.batch))
            for step in range(2):
                inputs = sess.step_inputs()
                outs = sess.alloc_outputs()
                outs.fill_(float("nan"))
                if mode == "calls":
                    for l in range(len(wl.layout)):
                        ent = inputs[l]
                        if "k" in ent:
                            sess.ctx.append_kv(l, ids, None, ent["k"], ent["v"])
                        sess.ctx.decode(l, ids, ent["q"], outs[l])
                    sess.pos += 1
                elif mode == "one":
                    sess.decode_step(inputs, outs)
                else:
                    sess.decode_step(inputs, outs, advance=False, layer_range=(0, 2))
                    sess.decode_step(inputs, outs, layer_range=(2, len(wl.layout)))
            torch.cuda.synchronize()
            assert sess.ctx.get_device_status() == 0
            state = [[sess.ctx.get_len(l, b) for b in ids] for l in range(len(wl.layout))]
            outs_by_mode.append((outs.clone(), state, [sess.ctx.get_block_table(b) for b in ids]))
        finally:
            sess.close()
    ref = outs_by_mode[0]
    for got in outs_by_mode[1:]:
        assert torch.equal(got[0].view(torch.int16), ref[0].view(torch.int16))
        assert got[1] == ref[1] and got[2] == ref[2]
