"""Rotary position embedding fused into the KV append, on a B200 against the CPU checker:
the stored key rows, and a decode step over rotated keys with rotated queries."""
import numpy as np
import pytest
import torch

from oracle import mixattn_oracle as mo
from synth import configs as cf
from synth import inputs as si

from gpu_common import check_close, load_lib, torch_dt

pytestmark = pytest.mark.gpu


def _round_to(x: np.ndarray, dtype):
    return torch.from_numpy(x).to(torch_dt(dtype)).double().numpy()


@pytest.mark.parametrize("dtype,D", [(cf.F32, 64), (cf.BF16, 128), (cf.BF16, 64)])
def test_rope_append_stores_rotated_keys_and_decode_matches(dtype, D):
    mx, runner = load_lib()
    theta = 500000.0
    n_ctx = 70000                     # positions far beyond 2 pi / (smallest frequency step)
    wl = cf.tiny_decode().scaled(batch=2, context=0, head_dim=D, dtype=dtype)
    sess = runner.Session(wl, [n_ctx, 300], headroom_tokens=2)
    dt = torch_dt(dtype)
    lens = [n_ctx, 300]
    try:
        # bulk append with the embedding fused, in two calls so that the second starts mid-sequence
        for o in cf.owners_of(wl.layout):
            for part in (0, 1):
                ks, vs, ns = [], [], []
                for b, n in enumerate(lens):
                    a, e = (0, n // 3) if part == 0 else (n // 3, n)
                    K, V = si.kv_tokens(wl.seed, o, b, a, e - a, wl.n_kv_heads, D, dt, "cuda")
                    ks.append(K)
                    vs.append(V)
                    ns.append(e - a)
                sess.ctx.append_kv_rope(o, [0, 1], ns, torch.cat(ks), torch.cat(vs), theta)
        torch.cuda.synchronize()
        assert sess.ctx.get_device_status() == 0
        # stored rows: keys rotated at their positions, values untouched
        ulp = 2.0 ** -8 if dtype == cf.BF16 else 2.0 ** -20      # bf16: one unit in the last place; fp32: a few
        for l in (0, 1):
            kind, W, owner = wl.layout[l]
            for b, n in enumerate(lens):
                lo = 0 if kind == cf.FULL else n - W
                for pos in sorted({lo, lo + 1, (lo + n) // 2, n - 2, n - 1}):
                    K, V = si.kv_tokens(wl.seed, owner, b, pos, 1, wl.n_kv_heads, D, dt)
                    kr = mo.rope_rotate(K, [pos], theta)[0]
                    gk, gv = sess.ctx.debug_read_kv(l, b, pos)
                    assert torch.equal(gv.view(torch.int16 if dtype == cf.BF16 else torch.int32),
                                       V[0].view(torch.int16 if dtype == cf.BF16 else torch.int32))
                    err = np.abs(gk.double().numpy() - kr)
                    # fp32 rotation of dtype inputs, rounded once: within one unit of the pair's magnitude
                    mag = np.repeat(np.hypot(kr[:, 0::2], kr[:, 1::2]), 2, axis=1)
                    assert (err <= ulp * np.maximum(mag, 1e-3)).all(), f"layer {l} seq {b} pos {pos}: {err.max():.3e}"
        # one decode step: a plain append of an already rotated key, then rotated queries over the cache
        ids = [0, 1]
        for l, (kind, W, owner) in enumerate(wl.layout):
            if owner == l:
                ks, vs = [], []
                for b, n in enumerate(lens):
                    K, V = si.kv_tokens(wl.seed, l, b, n, 1, wl.n_kv_heads, D, dt, "cuda")
                    ks.append(K)
                    vs.append(V)
                sess.ctx.append_kv_rope(l, ids, None, torch.cat(ks), torch.cat(vs), theta)
            qs = []
            for b, n in enumerate(lens):
                q = si.q_tokens(wl.seed, l, b, n, 1, wl.n_q_heads, D, dt)
                qs.append(torch.from_numpy(mo.rope_rotate(q, [n], theta)).to(dt))
            q = torch.cat(qs).cuda()
            out = torch.empty_like(q)
            sess.ctx.decode(l, ids, q, out)
            torch.cuda.synchronize()
            got = out.float().cpu().double().numpy()
            for b, n in enumerate(lens):
                lo = 0 if kind == cf.FULL else max(0, n + 1 - W)
                K, V = si.kv_tokens(wl.seed, owner, b, lo, n + 1 - lo, wl.n_kv_heads, D, dt)
                Kr = _round_to(mo.rope_rotate(K, np.arange(lo, n + 1), theta), dtype)
                ref = mo.decode_attention(qs[b][0], Kr, V, cf.FULL, 0)
                check_close(got[b], ref, dtype, f"decode over rotated keys, layer {l} seq {b}")
        assert sess.ctx.rc_append_kv_rope(0, ids, None, q, q, 1.0) == mx.ERR_INVALID_ARG
        assert sess.ctx.rc_append_kv_rope(3, ids, None, q, q, theta) == mx.ERR_NOT_OWNER
    finally:
        sess.close()
