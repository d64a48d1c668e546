"""Host-side cache bookkeeping through the C ABI (host-only contexts, no GPU),
bit-exact against the CPU checker's integer simulation; error paths; exports."""
import os
import re

import numpy as np
import pytest

from oracle import mixattn_oracle as mo
from synth import configs as cf
from paper_2409_15012_b200 import build as mbuild

mbuild.build()
from paper_2409_15012_b200 import binding as mx  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "mixattn.h")).read()
    declared = set(re.findall(r"\b(mixattn_[a-z0-9_]+)\s*\(", text))
    assert declared, "no declarations parsed"
    for name in declared:
        assert hasattr(mx.lib, name), name
    assert declared == set(mx.EXPORTS)
    assert mx.strerror(0) == "ok" and "page" in mx.strerror(mx.ERR_OUT_OF_PAGES)
    assert mx.strerror(-99) == "unknown status"


def _compare_state(ctx, ph, layout, B):
    assert ctx.get_n_free_pages() == ph.n_free_pages()
    for b in range(B):
        assert ctx.get_block_table(b) == ph.get_block_table(b)
        for l, (kind, W, owner) in enumerate(layout):
            n = ph.get_len(l, b)
            assert ctx.get_len(l, b) == n
            if kind == mo.SLIDING:
                assert ctx.get_ring_state(l, b) == ph.get_ring_state(l, b)
            for pos in {0, n // 2, n - 1, n - W, n - W - 1} if kind == mo.SLIDING else {0, n // 2, n - 1}:
                try:
                    want = ph.locate(l, b, pos)
                except mo.OracleError:
                    want = None
                a, s = mx.C.c_int32(), mx.C.c_int32()
                rc = mx.lib.mixattn_locate(ctx.h, l, b, pos, mx.C.byref(a), mx.C.byref(s))
                if want is None:
                    assert rc == mx.ERR_INVALID_ARG
                else:
                    assert rc == 0 and (a.value, s.value) == want


@pytest.mark.parametrize("layout_name", ["tiny", "mid6", "pairs8", "two_full"])
def test_bookkeeping_matches_checker_bit_exactly(layout_name):
    layout = {
        "tiny": cf.layout_tiny(5),
        "mid6": cf.layout_mid(7, 6),
        "pairs8": cf.layout_pairs(4, 8),
        "two_full": [(0, 0, 0), (0, 0, 1), (1, 3, 2), (0, 0, 1)],
    }[layout_name]
    B, n_pages = 5, 40
    rng = np.random.default_rng(hash(layout_name) % 1000)
    perm = rng.permutation(n_pages).astype(np.int32)
    ctx = mx.Context(layout, 4, 2, 64, mx.F32, B, n_pages, free_order=perm, device=-1)
    ph = mo.PhysicalCache(layout, 2, 64, B, n_pages, free_order=perm, store_values=False)
    owners = cf.owners_of(layout)
    for step in range(120):
        op = rng.integers(0, 10)
        if op == 0:
            b = int(rng.integers(0, B))
            ctx.seq_reset(b)
            ph.seq_reset(b)
        else:
            ids = rng.permutation(B)[: rng.integers(1, B + 1)].tolist()
            n_new = None if op < 6 else rng.integers(0, 40, size=len(ids)).tolist()
            for o in owners:
                rc = ctx.rc_append_kv(o, ids, n_new)
                try:
                    ph.append(o, ids, n_new)
                    want = 0
                except mo.OracleError as e:
                    want = e.code
                assert rc == want, (step, o, rc, want)
        _compare_state(ctx, ph, layout, B)
    ctx.close()


def test_error_paths_change_nothing():
    layout = cf.layout_tiny(4)
    ctx = mx.Context(layout, 4, 2, 64, mx.F32, 2, 3, device=-1)
    assert ctx.rc_append_kv(2, [0]) == mx.ERR_NOT_OWNER
    assert ctx.rc_append_kv(3, [0]) == mx.ERR_NOT_OWNER
    assert ctx.rc_append_kv(0, [2]) == mx.ERR_BAD_SEQ
    assert ctx.rc_append_kv(0, [0, 0]) == mx.ERR_INVALID_ARG
    assert ctx.rc_append_kv(9, [0]) == mx.ERR_INVALID_ARG
    assert ctx.rc_append_kv(0, [0], [-1]) == mx.ERR_INVALID_ARG
    assert ctx.rc_decode(0, [0], None, None) == mx.ERR_INVALID_ARG        # null q/out
    ctx.append_kv(0, [0], [33])
    assert ctx.rc_append_kv(0, [0, 1], [1, 1]) == mx.ERR_OUT_OF_PAGES
    assert ctx.get_len(0, 0) == 33 and ctx.get_len(0, 1) == 0 and ctx.get_n_free_pages() == 0
    assert ctx.rc_append_kv(0, [0], [100]) == mx.ERR_INVALID_ARG          # beyond max_seq_len (48)
    # host-only context: the GPU calls say so, after validating
    import ctypes
    dummy = ctypes.c_void_p(256)
    s = np.array([1], dtype=np.int32)
    rc = mx.lib.mixattn_decode(ctx.h, 0, 1, mx._p32(s), dummy, dummy, None)
    assert rc == mx.ERR_EMPTY_CONTEXT
    s = np.array([0], dtype=np.int32)
    assert mx.lib.mixattn_decode(ctx.h, 0, 1, mx._p32(s), dummy, dummy, None) == mx.ERR_CUDA
    with pytest.raises(mx.MixAttnError):
        ctx.get_ring_state(0, 0)
    ctx.close()


def test_create_rejects_bad_layouts_and_fields():
    bad_layouts = [
        [(0, 0, 1), (0, 0, 1)],
        [(0, 0, 0), (0, 0, 0), (0, 0, 1)],
        [(0, 0, 0), (1, 4, 0)],
        [(1, 4, 0), (1, 8, 0)],
        [(1, 0, 0)],
        [(2, 0, 0)],
        [],
    ]
    for lay in bad_layouts:
        with pytest.raises(mx.MixAttnError) as e:
            mx.Context(lay, 4, 2, 64, mx.F32, 2, 4, device=-1)
        assert e.value.code == mx.ERR_INVALID_LAYOUT, lay
        with pytest.raises(mo.OracleError):
            mo.validate_layout(lay)
    ok = cf.layout_tiny()
    for kw in (dict(n_q_heads=5), dict(head_dim=96), dict(dtype=3), dict(max_seqs=0)):
        args = dict(n_q_heads=4, n_kv_heads=2, head_dim=64, dtype=mx.F32, max_seqs=2, n_pages=4)
        args.update(kw)
        with pytest.raises(mx.MixAttnError) as e:
            mx.Context(ok, device=-1, **args)
        assert e.value.code == mx.ERR_INVALID_ARG
    cfg, keep = mx.make_config(ok, 4, 2, 64, mx.F32, 2, 4, page_size=32)
    with pytest.raises(mx.MixAttnError):
        mx.arena_bytes(cfg)
    cfg, keep = mx.make_config(ok, 4, 2, 64, mx.F32, 2, 4, free_order=[0, 1, 1, 3])
    with pytest.raises(mx.MixAttnError):
        mx.arena_bytes(cfg)


def test_cache_bytes_follow_the_sharing_law():
    Hkv, D, B, n_pages = 8, 128, 4, 100
    for dtype, e in ((mx.BF16, 2), (mx.F32, 4)):
        for lay in (cf.layout_mid(1024), cf.layout_pairs(1024), cf.layout_all_full(3),
                    [(0, 0, 0)] * 3, cf.layout_all_sliding(2, 64)):
            cfg, keep = mx.make_config(lay, 32, Hkv, D, dtype, B, n_pages)
            ph = mo.PhysicalCache(lay, Hkv, D, B, n_pages, store_values=False)
            assert mx.cache_bytes(cfg) == ph.cache_bytes(e)
            assert mx.arena_bytes(cfg) > mx.cache_bytes(cfg)


def test_chunk_and_rope_calls_on_a_host_only_context():
    # argument checks run on the host before anything else; a host-only context keeps the
    # bookkeeping of a rope append (k / v ignored) and cannot attend
    layout = cf.layout_tiny(8)
    ph = mo.PhysicalCache(layout, 2, 64, 2, 6, store_values=False)
    ctx = mx.Context(layout, 4, 2, 64, mx.F32, 2, 6, device=-1)
    assert ctx.rc_attend_chunk(0, [0], [4], None, None, None, None) == mx.ERR_UNSUPPORTED   # no scratch configured
    ctx.close()
    ctx = mx.Context(layout, 4, 2, 64, mx.F32, 2, 6, device=-1, chunk_scratch_tokens=32)
    for o in cf.owners_of(layout):
        assert ctx.rc_append_kv_rope(o, [0, 1], [20, 3], None, None, 10000.0) == 0
        ph.append(o, [0, 1], [20, 3])
    _compare_state(ctx, ph, layout, 2)
    assert ctx.rc_append_kv_rope(0, [0], [1], None, None, 1.0) == mx.ERR_INVALID_ARG        # theta must exceed 1
    assert ctx.rc_append_kv_rope(0, [0], [1], None, None, float("inf")) == mx.ERR_INVALID_ARG
    assert ctx.rc_append_kv_rope(2, [0], [1], None, None, 10000.0) == mx.ERR_NOT_OWNER
    assert ctx.rc_attend_chunk(0, [0, 0], [1, 1], None, None, None, None) == mx.ERR_INVALID_ARG
    assert ctx.rc_attend_chunk(0, [5], [1], None, None, None, None) == mx.ERR_BAD_SEQ
    assert ctx.rc_attend_chunk(0, [0], [0], None, None, None, None) == mx.ERR_INVALID_ARG
    assert ctx.rc_attend_chunk(7, [0], [1], None, None, None, None) == mx.ERR_INVALID_ARG
    assert ctx.rc_attend_chunk(0, [0], [13], None, None, None, None) == mx.ERR_TOO_LARGE      # 20 cached + 13 > 32
    assert ctx.rc_attend_chunk(1, [0], [26], None, None, None, None) == mx.ERR_TOO_LARGE      # ring: 7 cached + 26 > 32
    assert ctx.rc_attend_chunk(1, [0], [25], None, None, None, None) == mx.ERR_CUDA           # fits; no device
    assert ctx.rc_attend_chunk(0, [0, 1], [4, 4], None, None, None, None) == mx.ERR_CUDA
    _compare_state(ctx, ph, layout, 2)                                                        # nothing stored
    # the switch for sharing one copy among the layers of a cache is host state: settable without a
    # device, and it changes no check above
    assert mx.lib.mixattn_set_chunk_gather_reuse(None, 1) == mx.ERR_INVALID_ARG
    assert mx.lib.mixattn_set_chunk_ring_direct(None, 1) == mx.ERR_INVALID_ARG
    ctx.set_chunk_ring_direct(False)
    ctx.set_chunk_ring_direct(True)
    ctx.set_chunk_gather_reuse(True)
    assert ctx.rc_attend_chunk(0, [0], [13], None, None, None, None) == mx.ERR_TOO_LARGE
    assert ctx.rc_attend_chunk(1, [0], [25], None, None, None, None) == mx.ERR_CUDA
    ctx.set_chunk_gather_reuse(False)
    ctx.close()


def test_quantised_storage_config_rules_and_cache_bytes():
    # quantised KV storage needs bf16 I/O and head_dim 128; it stores head_dim + 1 bytes per head vector
    lay = cf.layout_mid(1024)
    ok = mx.make_config(lay, 32, 8, 128, mx.BF16, 4, 100, kv_format=mx.KV_FP8_E4M3)[0]
    native = mx.make_config(lay, 32, 8, 128, mx.BF16, 4, 100)[0]
    assert mx.cache_bytes(ok) * 2 * 128 == mx.cache_bytes(native) * 129
    for bad in (mx.make_config(lay, 32, 8, 128, mx.F32, 4, 100, kv_format=mx.KV_FP8_E4M3),
                mx.make_config(lay, 32, 8, 64, mx.BF16, 4, 100, kv_format=mx.KV_FP8_E4M3)):
        with pytest.raises(mx.MixAttnError) as ei:
            mx.cache_bytes(bad[0])
        assert ei.value.code == mx.ERR_UNSUPPORTED
    with pytest.raises(mx.MixAttnError) as ei:
        mx.cache_bytes(mx.make_config(lay, 32, 8, 128, mx.BF16, 4, 100, kv_format=7)[0])
    assert ei.value.code == mx.ERR_INVALID_ARG
    # a host-only quantised context keeps the same bookkeeping
    ctx = mx.Context(lay, 32, 8, 128, mx.BF16, 4, 100, device=-1, kv_format=mx.KV_FP8_E4M3)
    ctx.append_kv(0, [0, 1], [20, 3])
    assert ctx.get_len(12, 0) == 20 and ctx.get_block_table(0) == [0, 1] and ctx.get_block_table(1) == [2]
    ctx.close()


def test_decode_layers_stops_at_the_first_failing_call_and_says_where():
    import ctypes as C
    lay = cf.layout_tiny(64)
    ctx = mx.Context(lay, 4, 2, 64, mx.F32, 2, 8, device=-1)
    tab = (C.c_void_p * 4)(*([256] * 4))     # (never dereferenced: a host-only context launches nothing)
    # a host-only context keeps the books but cannot attend: layer 0's append stands, its decode fails
    rc, done = ctx.rc_decode_layers(0, 4, [0, 1], tab, tab, tab, tab)
    assert rc == mx.ERR_CUDA and done == 0
    assert ctx.get_len(0, 0) == 1 and ctx.get_len(1, 0) == 0
    # an empty range does nothing; bad ranges are refused
    assert ctx.rc_decode_layers(2, 2, [0], tab, tab, tab, tab) == (0, 0)
    assert ctx.rc_decode_layers(3, 2, [0], tab, tab, tab, tab)[0] == mx.ERR_INVALID_ARG
    assert ctx.rc_decode_layers(0, 5, [0], tab, tab, tab, tab)[0] == mx.ERR_INVALID_ARG
    assert ctx.rc_decode_layers(0, 1, [0], None, tab, tab, tab)[0] == mx.ERR_INVALID_ARG
    # a bad sequence id is refused by the first call, nothing moves
    rc, done = ctx.rc_decode_layers(1, 3, [7], tab, tab, tab, tab)
    assert rc == mx.ERR_BAD_SEQ and done == 0 and ctx.get_len(1, 0) == 0
    ctx.close()
