"""mixattn_decode_static_scratch against mixattn_decode.

Some users of the library cannot give it a workspace or allocate device memory
around the attention call (an engine that has handed out all its memory, a
buffer sized for the caches only, an allocator that must not be re-entered).
For them the library has a decode entry point whose split-KV partial results
live in a static device array.  This test drives that entry point through the
C ABI on a cache with several splits per sequence, twice in a row (the array
keeps the first call's contents), and requires the outputs of mixattn_decode:
within the bf16 tolerance of the other GPU tests, and, because both entry
points share one split planner and so add the partial results in the same
order, bit for bit.  The device's free-memory figure must be the same before
and after the call (nothing was allocated), and an oversized request must be
refused without a launch.

The file name sorts last on purpose: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest
import torch

from synth import configs as cf

from gpu_common import TOL, load_lib

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_decode_twice():
    mx, runner = load_lib()
    wl = cf.mid_decode().scaled(layout=cf.layout_tiny(512), batch=3, context=6000)
    sess = runner.Session(wl, [6000, 3000, 40], headroom_tokens=4)
    try:
        sess.fill(700)
        sess.ctx.set_split_tokens(256)            # several splits per sequence -> the scratch is used
        ids = list(range(wl.batch))
        tol = TOL[wl.dtype]
        for call in range(2):
            inputs = sess.step_inputs()
            for l in range(len(wl.layout)):
                ent = inputs[l]
                if "k" in ent:
                    sess.ctx.append_kv(l, ids, None, ent["k"], ent["v"])
                ref = torch.full((wl.batch, wl.n_q_heads, wl.head_dim), float("nan"),
                                 dtype=torch.bfloat16, device="cuda")
                got = torch.full_like(ref, float("nan"))
                sess.ctx.decode(l, ids, ent["q"], ref)
                launches = sess.ctx.get_launch_count()
                torch.cuda.synchronize()
                free_before = torch.cuda.mem_get_info()[0]
                rc = sess.ctx.rc_decode_static_scratch(l, ids, ent["q"], got)
                assert rc == 0, mx.strerror(rc)
                assert sess.ctx.get_launch_count() - launches == 2      # split pass + combine pass
                torch.cuda.synchronize()
                if call > 0 or l > 0:   # (the very first call may load the kernels' module)
                    assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
                a, b = got.float().cpu().numpy(), ref.float().cpu().numpy()
                assert np.isfinite(a).all()
                err = np.abs(a - b)
                assert err.max() <= tol["max_abs"] and err.mean() <= tol["mean_abs"], (call, l, err.max())
                assert torch.equal(got.view(torch.int16), ref.view(torch.int16)), (call, l, "bits differ")
            sess.pos += 1
        assert sess.ctx.get_device_status() == 0

        # a request that needs more than the 8 MiB array is refused, nothing is launched
        sess.ctx.set_split_tokens(16)
        q = inputs[0]["q"]
        out = torch.full_like(q, 3.0)
        launches = sess.ctx.get_launch_count()
        need = sum(-(-int(n) // 16) for n in sess.pos) * wl.n_q_heads * (wl.head_dim + 2) * 4
        assert need > 8 << 20
        assert sess.ctx.rc_decode_static_scratch(0, ids, q, out) == mx.ERR_TOO_LARGE
        assert sess.ctx.get_launch_count() == launches
        torch.cuda.synchronize()
        assert (out == 3.0).all()
        assert "scratch" in mx.strerror(mx.ERR_TOO_LARGE)
    finally:
        sess.close()
