"""Chunks of new tokens behind a cached prefix (chunked prompts, multi-token decode
steps) on a B200 against the CPU checker: every chunk of every layer element by element,
the cache state bit for bit after the appends that follow, and a decode step at the end."""
import numpy as np
import pytest
import torch

from oracle import mixattn_oracle as mo
from synth import configs as cf
from synth import inputs as si

from gpu_common import check_close, check_stored_bits, compare_state, load_lib, ref_decode, torch_dt

pytestmark = pytest.mark.gpu


def run_chunked(wl: cf.Workload, schedule, scratch: int, rows_per_chunk=None, ring_direct=True):
    """schedule[b] = chunk lengths of sequence b (0 = the sequence sits that round out)."""
    mx, runner = load_lib()
    B = wl.batch
    totals = [sum(s) for s in schedule]
    sess = runner.Session(wl, totals, headroom_tokens=2, chunk_scratch_tokens=scratch)
    ph = mo.PhysicalCache(wl.layout, wl.n_kv_heads, wl.head_dim, B, sess.n_pages, store_values=False)
    dt = torch_dt(wl.dtype)
    pos = [0] * B
    try:
        sess.ctx.set_chunk_ring_direct(ring_direct)
        for rnd in range(max(len(s) for s in schedule)):
            ids = [b for b in range(B) if rnd < len(schedule[b]) and schedule[b][rnd] > 0]
            lens = [schedule[b][rnd] for b in ids]
            if not ids:
                continue
            for l, (kind, W, owner) in enumerate(wl.layout):
                q = torch.cat([si.q_tokens(wl.seed, l, b, pos[b], n, wl.n_q_heads, wl.head_dim, dt)
                               for b, n in zip(ids, lens)])
                kv = [si.kv_tokens(wl.seed, owner, b, pos[b], n, wl.n_kv_heads, wl.head_dim, dt)
                      for b, n in zip(ids, lens)]
                k, v = torch.cat([a for a, _ in kv]), torch.cat([c for _, c in kv])
                out = torch.full_like(q, float("nan"), device="cuda")
                sess.ctx.attend_chunk(l, ids, lens, q.cuda(), k.cuda(), v.cuda(), out)
                torch.cuda.synchronize()
                got = out.float().cpu().double().numpy()
                row = 0
                for b, n in zip(ids, lens):
                    # the checker gets the whole history regenerated from the seed
                    Kh, Vh = si.kv_tokens(wl.seed, owner, b, 0, pos[b] + n, wl.n_kv_heads, wl.head_dim, dt)
                    rows = None
                    if rows_per_chunk is not None and n > rows_per_chunk:
                        rows = sorted(set(np.linspace(0, n - 1, rows_per_chunk).astype(int).tolist()))
                    ref = mo.prefill_attention(q[row:row + n], Kh, Vh, kind, W, prefix_len=pos[b], rows=rows)
                    g = got[row:row + n] if rows is None else got[row:row + n][rows]
                    check_close(g, ref, wl.dtype, f"round {rnd} layer {l} seq {b} prefix {pos[b]} chunk {n}")
                    row += n
            # every layer has seen the chunk: now the owners store it
            for o in cf.owners_of(wl.layout):
                kv = [si.kv_tokens(wl.seed, o, b, pos[b], n, wl.n_kv_heads, wl.head_dim, dt)
                      for b, n in zip(ids, lens)]
                k, v = torch.cat([a for a, _ in kv]).cuda(), torch.cat([c for _, c in kv]).cuda()
                sess.ctx.append_kv(o, ids, lens, k, v)
                ph.append(o, ids, lens)
            for b, n in zip(ids, lens):
                pos[b] += n
            torch.cuda.synchronize()
            compare_state(sess.ctx, ph, wl)
        assert sess.ctx.get_device_status() == 0
        sess.pos[:] = pos
        for l, (kind, W, owner) in enumerate(wl.layout):
            for b in range(B):
                lo = 0 if kind == cf.FULL else max(0, pos[b] - W)
                check_stored_bits(sess.ctx, ph, wl, l, b, sorted({lo, pos[b] - 1, (lo + pos[b]) // 2}))
        inputs = sess.step_inputs()
        outs = sess.alloc_outputs()
        sess.decode_step(inputs, outs)
        torch.cuda.synchronize()
        got = outs.float().cpu().double().numpy()
        for l in range(len(wl.layout)):
            for b in range(B):
                check_close(got[l, b], ref_decode(wl, l, b, pos[b] + 1), wl.dtype, f"decode after chunks {l}/{b}")
    finally:
        sess.close()


def test_chunks_fp32_tiny_layout():
    # window 64: chunks shorter than, equal to and longer than the window, single tokens, a
    # sequence that joins late, and a scratch that only holds one sequence's keys at the end
    wl = cf.tiny_decode().scaled(batch=3, context=0)
    schedule = [[100, 1, 37, 64, 200, 1], [5, 64, 129, 3, 0, 70], [0, 0, 300, 1, 1, 33]]
    run_chunked(wl, schedule, scratch=640)


@pytest.mark.parametrize("ring_direct", [True, False])
def test_chunks_bf16_tensor_core_path(ring_direct):
    # head_dim 128, bf16: the tcgen05 kernel with a key prefix that is not a multiple of the
    # tile (diagonal inside tiles), window 256 shared by a reader, several query tiles; with the
    # rings read in place and with every cached key copied first
    wl = cf.prefill_chunk().scaled(layout=cf.layout_tiny(256), batch=2, seq_len=0)
    schedule = [[300, 129, 1, 500, 77], [50, 700, 128, 4, 256]]
    run_chunked(wl, schedule, scratch=2600, ring_direct=ring_direct)


def test_chunks_bf16_mid_layout_sampled_rows():
    # the 24-layer layout (two shared rings of 1024 read in place, one shared paged cache whose
    # keys are copied), longer prefixes
    wl = cf.prefill_chunk().scaled(batch=2, seq_len=0)
    schedule = [[1500, 1100, 130], [900, 2048, 1]]
    run_chunked(wl, schedule, scratch=6000, rows_per_chunk=24)


@pytest.mark.parametrize("window", [128, 384])
def test_chunks_read_the_ring_in_place_at_every_kind_of_prefix(window):
    # cached lengths that end on a tile edge, one token before and after it, inside the first
    # tile, exactly at the window, and several turns of the ring later; chunks of one token, of
    # less than a tile, of a tile and of several; three sequences at different offsets in one call
    wl = cf.prefill_chunk().scaled(layout=cf.layout_tiny(window), batch=3, seq_len=0)
    schedule = [[1, 126, 1, 1, 127, window - 1, 1, 2 * window + 77, 130, 5],
                [128, 128, 1, window, 3, 0, 700, 1, 255, 256],
                [0, 127, 2, 0, 129, 64, 64, 64, 1000, 1]]
    run_chunked(wl, schedule, scratch=4096)


def test_chunks_bf16_head_dim_64():
    # 64-channel heads: rings read in place (pages of 16 x 128-byte rows), paged caches copied
    wl = cf.prefill_chunk().scaled(layout=cf.layout_tiny(256), batch=2, seq_len=0, n_q_heads=8, n_kv_heads=2, head_dim=64)
    run_chunked(wl, [[300, 129, 1, 500, 77], [50, 700, 128, 4, 256]], scratch=2600)


def test_chunk_window_not_a_multiple_of_the_tile_still_copies():
    # window 200: not a whole number of key tiles, so the call copies whatever the switch says
    wl = cf.prefill_chunk().scaled(layout=cf.layout_tiny(200), batch=2, seq_len=0)
    run_chunked(wl, [[300, 129, 1, 200], [50, 500, 128, 4]], scratch=2600, ring_direct=True)


def test_chunk_errors():
    mx, runner = load_lib()
    wl = cf.tiny_decode().scaled(batch=2, context=0)
    q = torch.zeros(8, wl.n_q_heads, wl.head_dim, device="cuda")
    kv = torch.zeros(8, wl.n_kv_heads, wl.head_dim, device="cuda")
    out = torch.full_like(q, 7.0)
    sess = runner.Session(wl, [40, 40], headroom_tokens=2)                      # no scratch
    try:
        assert sess.ctx.rc_attend_chunk(0, [0], [8], q, kv, kv, out) == mx.ERR_UNSUPPORTED
    finally:
        sess.close()
    sess = runner.Session(wl, [40, 40], headroom_tokens=2, chunk_scratch_tokens=16)
    try:
        sess.fill()
        assert sess.ctx.rc_attend_chunk(0, [0], [2], q, kv, kv, out) == mx.ERR_TOO_LARGE   # 40 cached + 2 > 16
        assert sess.ctx.rc_attend_chunk(1, [0], [2], q, kv, kv, out) == mx.ERR_TOO_LARGE   # ring (window 64): 40 + 2 too
        assert sess.ctx.rc_attend_chunk(0, [0, 0], [1, 1], q, kv, kv, out) == mx.ERR_INVALID_ARG
        assert sess.ctx.rc_attend_chunk(0, [0], [0], q, kv, kv, out) == mx.ERR_INVALID_ARG
        assert sess.ctx.rc_attend_chunk(0, [2], [1], q, kv, kv, out) == mx.ERR_BAD_SEQ
        assert sess.ctx.rc_attend_chunk(0, [0], [3], q, kv, kv, out) == mx.ERR_INVALID_ARG  # beyond max_seq_len
        torch.cuda.synchronize()
        assert (out == 7.0).all()
        assert sess.ctx.get_len(0, 0) == 40                                             # nothing stored
    finally:
        sess.close()


def test_serving_trace_small():
    # prompts of different lengths served in chunks, then decode steps, through the runner's
    # helpers; the cache state and the last step's outputs against the checker
    mx, runner = load_lib()
    wl = cf.mid_decode().scaled(layout=cf.layout_mid(128, 6), batch=3, context=0, n_q_heads=12, n_kv_heads=3)
    prompts = [700, 333, 129]
    sess = runner.Session(wl, prompts, headroom_tokens=6, chunk_scratch_tokens=3 * (700 + 256))
    ph = mo.PhysicalCache(wl.layout, wl.n_kv_heads, wl.head_dim, wl.batch, sess.n_pages, store_values=False)
    sess.mirror = ph
    try:
        outs = sess.prefill_in_chunks(256)
        torch.cuda.synchronize()
        compare_state(sess.ctx, ph, wl)
        assert [int(p) for p in sess.pos] == prompts
        # the last round held only sequence 0's final 188 tokens: check its last row in every layer
        dt = torch_dt(wl.dtype)
        for l, (kind, W, owner) in enumerate(wl.layout):
            q = si.q_tokens(wl.seed, l, 0, 699, 1, wl.n_q_heads, wl.head_dim, dt)
            Kh, Vh = si.kv_tokens(wl.seed, owner, 0, 0, 700, wl.n_kv_heads, wl.head_dim, dt)
            ref = mo.prefill_attention(q, Kh, Vh, kind, W, prefix_len=699)
            check_close(outs[l][-1:].float().cpu().double().numpy(), ref, wl.dtype, f"last prompt row, layer {l}")
        got = None
        for _ in range(5):
            o = sess.alloc_outputs()
            sess.decode_step(sess.step_inputs(), o)
            got = o
        torch.cuda.synchronize()
        compare_state(sess.ctx, ph, wl)
        g = got.float().cpu().double().numpy()
        for l in range(len(wl.layout)):
            for b in range(wl.batch):
                check_close(g[l, b], ref_decode(wl, l, b, prompts[b] + 5), wl.dtype, f"decode {l}/{b}")
        res = runner.serve_trace(wl.layout, 12, 3, 128, 2, 300, 3, 128)
        assert res["device_status"] == 0 and res["prefill_kernel_ms"] > 0 and res["decode_kernel_ms"] > 0
        # the same requests two at a time, the last wave only half full: same token count, three waves
        res = runner.serve_trace(wl.layout, 12, 3, 128, 5, 300, 3, 128, concurrency=2)
        assert res["device_status"] == 0 and res["waves"] == 3 and res["wall_tokens_per_s"] > 0
        assert res["tokens_per_s"] >= res["wall_tokens_per_s"]
    finally:
        sess.close()


@pytest.mark.parametrize("scratch_seqs,ring_direct", [(2, False), (1, False), (2, True)])
def test_gather_reuse_same_outputs_fewer_copies(scratch_seqs, ring_direct):
    # Layers that share a cache gather the same rows: with reuse enabled the copy runs once per run
    # of such layers (6-layer layout: standard owner, ring owner, two ring readers, a reader of the
    # standard cache, a second ring owner = 4 copies per round instead of 6) and every output is
    # bit-identical.  With a scratch that holds one sequence at a time the call works in two
    # pieces and must copy every time.  With the rings read in place only the two layers on the
    # standard cache copy, and the second of them finds the first one's rows still in the scratch.
    mx, runner = load_lib()
    layout = [(cf.FULL, 0, 0), (cf.SLIDING, 256, 1), (cf.SLIDING, 256, 1), (cf.SLIDING, 256, 1),
              (cf.FULL, 0, 0), (cf.SLIDING, 256, 5)]
    wl = cf.prefill_chunk().scaled(layout=layout, batch=2, seq_len=0)
    total, chunk = 900, 300
    results = []
    for reuse in (False, True):
        sess = runner.Session(wl, [total, total], headroom_tokens=2,
                              chunk_scratch_tokens=scratch_seqs * total if scratch_seqs == 2 else total + 8)
        try:
            sess.ctx.set_chunk_gather_reuse(reuse)
            sess.ctx.set_chunk_ring_direct(ring_direct)
            sess.ctx.profile_enable(True)
            outs = sess.prefill_in_chunks(chunk)
            torch.cuda.synchronize()
            n_gather = sess.ctx.profile_read(mx.K_GATHER)[0]
            sess.ctx.profile_enable(False)
            assert sess.ctx.get_device_status() == 0
            results.append(([o.clone() for o in outs], n_gather))
        finally:
            sess.close()
    (off, n_off), (on, n_on) = results
    for a, b in zip(off, on):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    rounds = total // chunk
    if ring_direct:
        assert n_off == 2 * rounds and n_on == 1 * rounds
    elif scratch_seqs == 2:
        assert n_off == 6 * rounds and n_on == 4 * rounds
    else:
        # the first round (empty caches, 2 x 300 rows) still fits in one piece; the later rounds
        # take two pieces per call and copy each time
        assert n_off == 6 + 12 * (rounds - 1) and n_on == 4 + 12 * (rounds - 1)
