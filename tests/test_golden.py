"""The stored results of the tiny fp32 decode configuration (tests/golden/tiny_decode_step.txt,
written by tests/golden/make_golden.py from the CPU checker alone).

CPU: the checker still reproduces the file (cache state exactly, outputs to 1e-12), and the file's
integer lines agree with what the rules give by hand for this case.  GPU: the library, through the
C ABI, reproduces the file (cache state exactly, outputs within the fp32 tolerance 1e-5)."""
import importlib.util
import os

import numpy as np
import pytest
import torch

from synth import configs as cf

GOLDEN_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
PATH = os.path.join(GOLDEN_DIR, "tiny_decode_step.txt")


def _load_script():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(GOLDEN_DIR, "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def _read():
    state, outs = [], {}
    with open(PATH) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w = line.split()
            if w[0] == "out":
                outs[(int(w[1]), int(w[2]), int(w[3]))] = np.array([float(x) for x in w[4:]])
            else:
                state.append(line)
    return state, outs


def test_checker_reproduces_the_stored_file():
    mg = _load_script()
    state, outs = mg.compute()
    g_state, g_outs = _read()
    assert state == g_state
    assert len(g_outs) == 4 * 2 * 4
    for (l, b, h), ref in g_outs.items():
        np.testing.assert_allclose(outs[(l, b)][h, :mg.CHANNELS], ref, rtol=0, atol=1e-12)


def test_stored_integers_follow_the_rules_by_hand():
    # 2 sequences filled 100 + 100 + 56 tokens, 16-token pages taken first-in first-out, sequence 0
    # before sequence 1 in every round: 7 + 6 + 3 pages each, then page 17 of each for token 256.
    state, _ = _read()
    s = dict((ln.split(" ", 1)[0] + " " + ln.split(" ", 2)[1], ln) for ln in state if ln.startswith("block_table"))
    t0 = [int(x) for x in s["block_table 0"].split()[2:]]
    t1 = [int(x) for x in s["block_table 1"].split()[2:]]
    assert t0 == list(range(0, 7)) + list(range(14, 20)) + [26, 27, 28] + [32]
    assert t1 == list(range(7, 14)) + list(range(20, 26)) + [29, 30, 31] + [33]
    # ring of 64 slots after 257 tokens: next slot 257 mod 64 = 1, all 64 valid; token 256 sits in slot 0
    assert "ring 1 0 1 64" in state and "ring 2 1 1 64" in state
    assert "locate 1 0 256 -1 0" in state and "locate 3 1 256 33 0" in state
    assert "free_pages 2" in state


@pytest.mark.gpu
def test_library_reproduces_the_stored_file():
    from gpu_common import load_lib
    _, runner = load_lib()
    wl = cf.tiny_decode()
    g_state, g_outs = _read()
    sess = runner.Session(wl, [wl.context] * wl.batch, headroom_tokens=1, n_pages=wl.batch * (wl.context // 16 + 2))
    try:
        sess.fill(100)
        inputs = sess.step_inputs()
        outs = sess.alloc_outputs()
        outs.fill_(float("nan"))
        sess.decode_step(inputs, outs)
        torch.cuda.synchronize()
        assert sess.ctx.get_device_status() == 0
        ctx = sess.ctx
        state = []
        for b in range(wl.batch):
            state.append(f"block_table {b} " + " ".join(str(p) for p in ctx.get_block_table(b)))
        for l, (kind, W, owner) in enumerate(wl.layout):
            for b in range(wl.batch):
                state.append(f"len {l} {b} {ctx.get_len(l, b)}")
                if kind == cf.SLIDING:
                    nxt, valid = ctx.get_ring_state(l, b)
                    state.append(f"ring {l} {b} {nxt} {valid}")
                page, slot = ctx.locate(l, b, wl.context)
                state.append(f"locate {l} {b} {wl.context} {page} {slot}")
        state.append(f"free_pages {ctx.get_n_free_pages()}")
        assert state == g_state
        got = outs.double().cpu().numpy()
        for (l, b, h), ref in g_outs.items():
            np.testing.assert_allclose(got[l, b, h, :ref.size], ref, rtol=0, atol=1e-5)
    finally:
        sess.close()
