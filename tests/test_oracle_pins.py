"""Pins for the CPU checker: brute force, a library routine, closed forms,
window-edge needles and the invariants the method must satisfy.  None of them
re-uses the checker's own formula: the brute force is a dense masked score
matrix with naive exponentials over repeated KV heads."""
import math

import numpy as np
import pytest
import torch

from oracle import mixattn_oracle as mo
from synth import configs as cf

FULL, SLIDING = mo.FULL, mo.SLIDING


def dense_reference(q, K, V, kind, window):
    """q [S,Hq,D], K,V [S,Hkv,D] -> [S,Hq,D]; mask matrix, no max subtraction."""
    S, Hq, D = q.shape
    G = Hq // K.shape[1]
    Kr = np.repeat(K, G, axis=1)        # head h uses KV head h // G
    Vr = np.repeat(V, G, axis=1)
    out = np.zeros((S, Hq, D))
    i = np.arange(S)[:, None]
    j = np.arange(S)[None, :]
    allowed = j <= i
    if kind == SLIDING:
        allowed &= (i - j) < window
    for h in range(Hq):
        sc = (q[:, h] @ Kr[:, h].T) / math.sqrt(D)
        w = np.where(allowed, np.exp(sc), 0.0)
        out[:, h] = (w / w.sum(axis=1, keepdims=True)) @ Vr[:, h]
    return out


def rnd(rng, *shape):
    return rng.standard_normal(shape)


@pytest.mark.parametrize("D", [8, 64])
@pytest.mark.parametrize("window", [1, 3, 16, 100])
@pytest.mark.parametrize("kind", [FULL, SLIDING])
def test_brute_force_prefill_and_decode(D, window, kind):
    rng = np.random.default_rng(D * 1000 + window)
    S, Hq, Hkv = 37, 4, 2
    q, K, V = rnd(rng, S, Hq, D), rnd(rng, S, Hkv, D), rnd(rng, S, Hkv, D)
    ref = dense_reference(q, K, V, kind, window)
    got = mo.prefill_attention(q, K, V, kind, window)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)
    # decode = the last row of the same definition, for every prefix length
    for n in (1, 2, window, window + 1, S):
        if 1 <= n <= S:
            d = mo.decode_attention(q[n - 1], K[:n], V[:n], kind, window)
            np.testing.assert_allclose(d, ref[n - 1], rtol=0, atol=1e-12)


def test_matches_torch_sdpa_when_window_covers_context():
    rng = np.random.default_rng(7)
    S, Hq, Hkv, D = 33, 6, 3, 16
    q, K, V = rnd(rng, S, Hq, D), rnd(rng, S, Hkv, D), rnd(rng, S, Hkv, D)
    G = Hq // Hkv
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(K).repeat_interleave(G, dim=1).permute(1, 0, 2)[None]
    tv = torch.from_numpy(V).repeat_interleave(G, dim=1).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    ref = ref[0].permute(1, 0, 2).numpy()
    for kind, window in ((FULL, 0), (SLIDING, S), (SLIDING, 10 * S)):
        got = mo.prefill_attention(q, K, V, kind, window)
        np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


def test_hand_computed_two_keys():
    # scores 0 and ln 3 -> weights 1/4 and 3/4 (scale fixed to 1)
    q = np.array([[1.0, 0.0]])
    K = np.array([[[0.0, 5.0]], [[math.log(3.0), -2.0]]])
    V = np.array([[[4.0, 0.0]], [[0.0, 8.0]]])
    out = mo.decode_attention(q, K, V, FULL, 0, scale=1.0)
    np.testing.assert_allclose(out, [[1.0, 6.0]], atol=1e-14)
    # default scale is 1/sqrt(D): scores 0 and ln(3)/sqrt(2)
    out = mo.decode_attention(q, K, V, FULL, 0)
    w = 3.0 ** (1 / math.sqrt(2))
    np.testing.assert_allclose(out, [[4.0 / (1 + w), 8.0 * w / (1 + w)]], atol=1e-14)


def test_closed_forms():
    rng = np.random.default_rng(11)
    n, Hq, Hkv, D, W = 29, 4, 2, 8, 5
    q, K, V = rnd(rng, Hq, D), rnd(rng, n, Hkv, D), rnd(rng, n, Hkv, D)
    # constant V rows -> that row, whatever Q, K and the mask are
    c = rnd(rng, D)
    Vc = np.broadcast_to(c, (n, Hkv, D)).copy()
    for kind in (FULL, SLIDING):
        out = mo.decode_attention(q, K, Vc, kind, W)
        np.testing.assert_allclose(out, np.broadcast_to(c, (Hq, D)), atol=1e-13)
    # Q = 0 -> arithmetic mean of the attended V rows
    z = np.zeros((Hq, D))
    G = Hq // Hkv
    full = mo.decode_attention(z, K, V, FULL, 0)
    slid = mo.decode_attention(z, K, V, SLIDING, W)
    for h in range(Hq):
        np.testing.assert_allclose(full[h], V[:, h // G].mean(axis=0), atol=1e-13)
        np.testing.assert_allclose(slid[h], V[n - W:, h // G].mean(axis=0), atol=1e-13)
    # window 1 -> the newest V row
    one = mo.decode_attention(q, K, V, SLIDING, 1)
    for h in range(Hq):
        np.testing.assert_allclose(one[h], V[n - 1, h // G], atol=1e-13)


def test_gqa_mapping_is_contiguous_groups():
    # V of KV head g is the constant g+1: head h must return h // G + 1
    n, Hq, Hkv, D = 9, 12, 3, 4
    rng = np.random.default_rng(5)
    q, K = rnd(rng, Hq, D), rnd(rng, n, Hkv, D)
    V = np.zeros((n, Hkv, D))
    for g in range(Hkv):
        V[:, g] = g + 1
    out = mo.decode_attention(q, K, V, FULL, 0)
    np.testing.assert_allclose(out[:, 0], np.arange(Hq) // 4 + 1, atol=1e-13)


def _needle(n, D, j, lam=40.0):
    """K with one dominant key at position j for the query e_0."""
    K = np.zeros((n, 1, D))
    K[j, 0, 0] = lam * math.sqrt(D)
    V = np.zeros((n, 1, D))
    V[:, 0, 0] = np.arange(n)
    q = np.zeros((1, D))
    q[0, 0] = 1.0
    return q, K, V


def test_window_edge_needle_decode():
    n, D, W = 50, 4, 7
    # key n-W is the oldest one inside the window: seen
    q, K, V = _needle(n, D, n - W)
    out = mo.decode_attention(q, K, V, SLIDING, W)
    assert abs(out[0, 0] - (n - W)) < 1e-9
    # key n-W-1 is just outside: the output is the plain mean of the window
    q, K, V = _needle(n, D, n - W - 1)
    out = mo.decode_attention(q, K, V, SLIDING, W)
    assert abs(out[0, 0] - np.arange(n - W, n).mean()) < 1e-9
    # a standard layer sees it
    out = mo.decode_attention(q, K, V, FULL, 0)
    assert abs(out[0, 0] - (n - W - 1)) < 1e-9


def test_window_edge_needle_prefill_rows():
    S, D, W = 24, 4, 8
    for i in (W - 1, W, W + 1):
        for j, seen in ((i - W + 1, True), (i - W, False)):
            if j < 0:
                continue
            q1, K, V = _needle(S, D, j)
            q = np.zeros((S, 1, D))
            q[:, 0, 0] = 1.0
            out = mo.prefill_attention(q, K, V, SLIDING, W, rows=[i])
            if seen:
                assert abs(out[0, 0, 0] - j) < 1e-9
            else:
                lo = max(0, i - W + 1)
                assert abs(out[0, 0, 0] - np.arange(lo, i + 1).mean()) < 1e-9


def test_key_range_counts_exactly_window_keys():
    for W in (1, 2, 16, 1024):
        for i in (0, 1, W - 1, W, W + 1, 5 * W + 3):
            lo, hi = mo.key_range(SLIDING, W, i)
            assert hi == i + 1 and hi - lo == min(i + 1, W)
            assert mo.key_range(FULL, W, i) == (0, i + 1)


# ---------------------------------------------------------------------------
# invariants between the logical and the physical half
# ---------------------------------------------------------------------------

def _run_both(layout, n_tokens, Hq=4, Hkv=2, D=8, B=2, n_pages=64, free_order=None, seed=3):
    rng = np.random.default_rng(seed)
    lg = mo.LogicalCache(layout, Hq, Hkv, D)
    ph = mo.PhysicalCache(layout, Hkv, D, B, n_pages, free_order=free_order)
    owners = cf.owners_of(layout)
    outs = []
    for t in range(n_tokens):
        step = {}
        for l in range(len(layout)):
            if l in owners:
                K, V = rnd(rng, B, Hkv, D), rnd(rng, B, Hkv, D)
                for b in range(B):
                    lg.append(l, b, K[b:b + 1], V[b:b + 1])
                ph.append(l, list(range(B)), None, K, V)
            q = rnd(rng, B, Hq, D)
            for b in range(B):
                a = lg.decode(l, b, q[b])
                p = ph.decode(l, b, q[b])
                np.testing.assert_allclose(p, a, rtol=0, atol=1e-12)
                step[(l, b)] = (q[b], a)
        outs.append(step)
    return lg, ph, outs


def test_ring_wraparound_equals_last_window_slice():
    W = 5
    layout = cf.layout_tiny(W)
    for n in (1, 4, 5, 6, 9, 10, 11, 23):
        lg, ph, _ = _run_both(layout, n)
        for layer in (1, 2):
            for b in range(2):
                Kp, Vp = ph.gather(layer, b)
                Kl, Vl = lg.history(layer, b)
                Kl, Vl = Kl[max(0, n - W):], Vl[max(0, n - W):]
                assert Kp.shape[0] == min(n, W)
                # same multiset of (K, V) rows: sort rows lexicographically
                a = np.concatenate([Kp, Vp], axis=-1).reshape(Kp.shape[0], -1)
                c = np.concatenate([Kl, Vl], axis=-1).reshape(Kl.shape[0], -1)
                assert np.array_equal(a[np.lexsort(a.T)], c[np.lexsort(c.T)])
                assert ph.get_ring_state(layer, b) == (n % W, min(n, W))
                for pos in range(max(0, n - W), n):
                    assert ph.locate(layer, b, pos) == (-1, pos % W)
                    k, v = ph.read_kv(layer, b, pos)
                    full_K, full_V = lg.history(layer, b)
                    assert np.array_equal(k, full_K[pos]) and np.array_equal(v, full_V[pos])


def test_reader_equals_recompute_with_owner_history():
    layout = cf.layout_tiny(6)
    lg, ph, outs = _run_both(layout, 19)
    # layer 3 reads layer 0's cache, layer 2 reads layer 1's ring
    for reader, owner in ((3, 0), (2, 1)):
        kind, W, _ = layout[reader]
        for b in range(2):
            q, got = outs[-1][(reader, b)]
            K, V = lg.hist[(owner, b)]
            np.testing.assert_allclose(got, mo.decode_attention(q, K, V, kind, W), atol=1e-13)
    assert (3, 0) not in lg.hist and (2, 0) not in lg.hist      # readers store nothing


def test_window_at_least_context_equals_full():
    rng = np.random.default_rng(9)
    n, Hq, Hkv, D = 21, 4, 2, 8
    q, K, V = rnd(rng, Hq, D), rnd(rng, n, Hkv, D), rnd(rng, n, Hkv, D)
    full = mo.decode_attention(q, K, V, FULL, 0)
    for W in (n, n + 1, 1000):
        np.testing.assert_array_equal(mo.decode_attention(q, K, V, SLIDING, W), full)
    assert not np.allclose(mo.decode_attention(q, K, V, SLIDING, n - 1), full)


def test_results_do_not_depend_on_page_permutation():
    layout = cf.layout_tiny(4)
    perm = np.random.default_rng(1).permutation(64)
    _, ph_a, outs_a = _run_both(layout, 40)
    _, ph_b, outs_b = _run_both(layout, 40, free_order=perm)
    assert ph_a.get_block_table(0) != ph_b.get_block_table(0)
    for sa, sb in zip(outs_a, outs_b):
        for key in sa:
            np.testing.assert_array_equal(sa[key][1], sb[key][1])


def test_reader_append_is_rejected_and_layout_validation():
    layout = cf.layout_tiny(4)
    ph = mo.PhysicalCache(layout, 2, 8, 2, 8)
    with pytest.raises(mo.OracleError) as e:
        ph.append(2, [0])
    assert e.value.code == mo.ERR_NOT_OWNER
    bad = [
        [(FULL, 0, 1), (FULL, 0, 1)],                    # owner later than reader
        [(FULL, 0, 0), (FULL, 0, 0), (FULL, 0, 1)],      # chain: layer 1 owns nothing
        [(FULL, 0, 0), (SLIDING, 4, 0)],                 # kind differs
        [(SLIDING, 4, 0), (SLIDING, 8, 0)],              # window differs
        [(SLIDING, 0, 0)],                               # window < 1
        [(2, 0, 0)],                                     # unknown kind
        [],
    ]
    for lay in bad:
        with pytest.raises(mo.OracleError) as e:
            mo.validate_layout(lay)
        assert e.value.code == mo.ERR_INVALID_LAYOUT
    for lay in (cf.layout_tiny(), cf.layout_mid(), cf.layout_pairs(), cf.layout_all_full(3),
                cf.layout_all_sliding(3, 7)):
        mo.validate_layout(lay)


def test_cache_size_law():
    Hkv, D, B, n_pages, e = 8, 128, 4, 100, 2
    per_tok = 2 * Hkv * D * e
    one = mo.PhysicalCache(cf.layout_all_full(1), Hkv, D, B, n_pages, store_values=False)
    assert one.cache_bytes(e) == n_pages * 16 * per_tok
    # l full layers sharing one cache store 1/l of what l private caches store
    for l in (2, 3, 6):
        share = mo.PhysicalCache([(FULL, 0, 0)] * l, Hkv, D, B, n_pages, store_values=False)
        priv = mo.PhysicalCache(cf.layout_all_full(l), Hkv, D, B, n_pages, store_values=False)
        assert share.cache_bytes(e) * l == priv.cache_bytes(e)
    # a window-s layer stores s tokens per sequence
    s = mo.PhysicalCache(cf.layout_all_sliding(1, 1024), Hkv, D, B, n_pages, store_values=False)
    assert s.cache_bytes(e) == B * 1024 * per_tok
    mid = mo.PhysicalCache(cf.layout_mid(1024), Hkv, D, B, n_pages, store_values=False)
    assert mid.cache_bytes(e) == n_pages * 16 * per_tok + 2 * B * 1024 * per_tok
    assert len(cf.owners_of(cf.layout_pairs(1024))) == 13


# ---------------------------------------------------------------------------
# integer rules of the paged cache, against closed forms worked out by hand
# ---------------------------------------------------------------------------

def test_fifo_paging_closed_form():
    # three sequences appended round-robin, one token each, identity free list:
    # sequence s receives page 3*k + s for its k-th logical block
    ph = mo.PhysicalCache(cf.layout_all_full(1), 1, 4, 3, 30, store_values=False)
    for t in range(16 * 4 + 1):
        ph.append(0, [0, 1, 2])
        for s in range(3):
            assert ph.get_len(0, s) == t + 1
            assert ph.get_block_table(s) == [3 * k + s for k in range(t // 16 + 1)]
            assert ph.locate(0, s, t) == (3 * (t // 16) + s, t % 16)
    assert ph.n_free_pages() == 30 - 15
    # reset returns pages to the tail in logical-block order
    ph.seq_reset(1)
    assert ph.get_len(0, 1) == 0 and ph.get_block_table(1) == []
    assert list(ph.free) == list(range(15, 30)) + [1, 4, 7, 10, 13]
    # a multi-token append pops pages in position order
    ph.append(0, [1], [40])
    assert ph.get_block_table(1) == [15, 16, 17]


def test_out_of_pages_changes_nothing():
    ph = mo.PhysicalCache(cf.layout_all_full(1), 1, 4, 2, 3, store_values=False)
    ph.append(0, [0], [33])                      # 3 pages
    with pytest.raises(mo.OracleError) as e:
        ph.append(0, [0, 1], [1, 1])             # seq 0 fits its page, seq 1 needs a 4th
    assert e.value.code == mo.ERR_OUT_OF_PAGES
    assert ph.get_len(0, 0) == 33 and ph.get_len(0, 1) == 0 and ph.n_free_pages() == 0
    with pytest.raises(mo.OracleError) as e:
        mo.decode_attention(np.zeros((1, 4)), np.zeros((0, 1, 4)), np.zeros((0, 1, 4)), FULL, 0)
    assert e.value.code == mo.ERR_EMPTY_CONTEXT


def test_two_full_owners_share_one_block_table():
    lay = [(FULL, 0, 0), (FULL, 0, 1)]
    ph = mo.PhysicalCache(lay, 1, 4, 1, 8, store_values=False)
    for t in range(20):
        ph.append(0, [0])
        ph.append(1, [0])
    assert ph.get_block_table(0) == [0, 1] and ph.n_free_pages() == 6
    assert ph.get_len(0, 0) == 20 and ph.get_len(1, 0) == 20


# --------------------------------------------------------------------------
# chunks of queries behind a cached prefix
# --------------------------------------------------------------------------

@pytest.mark.parametrize("kind,window", [(FULL, 0), (SLIDING, 1), (SLIDING, 5), (SLIDING, 16), (SLIDING, 100)])
def test_chunk_behind_prefix_is_the_dense_masked_reference(kind, window):
    # rows prefix..prefix+S-1 of the dense masked reference over the whole sequence, for chunk
    # boundaries before, at and after the window length, and a single-token chunk
    rng = np.random.default_rng(11 + window)
    n, Hq, Hkv, D = 41, 4, 2, 8
    q, K, V = rnd(rng, n, Hq, D), rnd(rng, n, Hkv, D), rnd(rng, n, Hkv, D)
    ref = dense_reference(q, K, V, kind, window)
    for prefix, S in ((0, n), (1, 40), (4, 9), (5, 1), (16, 25), (17, 3), (40, 1)):
        got = mo.prefill_attention(q[prefix:prefix + S], K[:prefix + S], V[:prefix + S], kind, window,
                                   prefix_len=prefix)
        np.testing.assert_allclose(got, ref[prefix:prefix + S], rtol=0, atol=1e-12)


def test_chunk_behind_prefix_matches_torch_sdpa_with_an_explicit_mask():
    rng = np.random.default_rng(5)
    prefix, S, Hq, Hkv, D, W = 13, 7, 6, 2, 16, 6
    n = prefix + S
    q, K, V = rnd(rng, S, Hq, D), rnd(rng, n, Hkv, D), rnd(rng, n, Hkv, D)
    G = Hq // Hkv
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(K).repeat_interleave(G, dim=1).permute(1, 0, 2)[None]
    tv = torch.from_numpy(V).repeat_interleave(G, dim=1).permute(1, 0, 2)[None]
    pos_q = torch.arange(prefix, n)[:, None]
    pos_k = torch.arange(n)[None, :]
    for kind, window, mask in ((FULL, 0, pos_k <= pos_q),
                               (SLIDING, W, (pos_k <= pos_q) & (pos_q - pos_k < W))):
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask)
        ref = ref[0].permute(1, 0, 2).numpy()
        got = mo.prefill_attention(q, K, V, kind, window, prefix_len=prefix)
        np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


def test_single_token_chunk_is_decode():
    rng = np.random.default_rng(9)
    n, Hq, Hkv, D = 30, 4, 1, 8
    q, K, V = rnd(rng, 1, Hq, D), rnd(rng, n, Hkv, D), rnd(rng, n, Hkv, D)
    for kind, window in ((FULL, 0), (SLIDING, 7)):
        a = mo.prefill_attention(q, K, V, kind, window, prefix_len=n - 1)[0]
        b = mo.decode_attention(q[0], K, V, kind, window)
        np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)


def test_chunk_needs_every_key_up_to_its_last_query():
    rng = np.random.default_rng(1)
    q, K = rnd(rng, 3, 2, 4), rnd(rng, 9, 2, 4)
    with pytest.raises(mo.OracleError):
        mo.prefill_attention(q, K, K, FULL, 0, prefix_len=5)


# --------------------------------------------------------------------------
# rotary position embedding
# --------------------------------------------------------------------------

def test_rope_is_complex_multiplication_by_unit_phases():
    # the same definition written with complex numbers: (x_2i + j x_2i+1) * exp(j m theta^(-2i/d))
    rng = np.random.default_rng(3)
    n, H, d, theta = 9, 2, 16, 10000.0
    x = rnd(rng, n, H, d)
    pos = np.array([0, 1, 2, 7, 100, 4095, 31999, 131071, 5])
    z = x[..., 0::2] + 1j * x[..., 1::2]
    freq = theta ** (-np.arange(0, d, 2) / d)
    zr = z * np.exp(1j * pos[:, None, None] * freq[None, None, :])
    got = mo.rope_rotate(x, pos, theta)
    np.testing.assert_allclose(got[..., 0::2], zr.real, rtol=0, atol=1e-9)
    np.testing.assert_allclose(got[..., 1::2], zr.imag, rtol=0, atol=1e-9)


def test_rope_closed_forms_and_relative_position_property():
    rng = np.random.default_rng(4)
    d, theta = 8, 500000.0
    q, k = rnd(rng, 1, 1, d), rnd(rng, 1, 1, d)
    # position 0 is the identity; the first pair turns by exactly m radians (theta^0 = 1)
    np.testing.assert_allclose(mo.rope_rotate(q, [0], theta), q, rtol=0, atol=0)
    e = np.zeros((1, 1, d)); e[0, 0, 0] = 1.0
    r = mo.rope_rotate(e, [3], theta)
    assert abs(r[0, 0, 0] - math.cos(3.0)) < 1e-15 and abs(r[0, 0, 1] - math.sin(3.0)) < 1e-15
    # the last pair turns by m * theta^(-(d-2)/d)
    e = np.zeros((1, 1, d)); e[0, 0, d - 2] = 1.0
    r = mo.rope_rotate(e, [1000], theta)
    a = 1000.0 * theta ** (-(d - 2) / d)
    assert abs(r[0, 0, d - 2] - math.cos(a)) < 1e-12 and abs(r[0, 0, d - 1] - math.sin(a)) < 1e-12
    # norms of pairs are kept; scores depend on the position difference only
    for m, n_ in ((5, 2), (1000, 997), (70000, 69997)):
        qm, kn = mo.rope_rotate(q, [m], theta), mo.rope_rotate(k, [n_], theta)
        np.testing.assert_allclose(np.hypot(qm[..., 0::2], qm[..., 1::2]), np.hypot(q[..., 0::2], q[..., 1::2]), atol=1e-12)
        ref = float((mo.rope_rotate(q, [m - n_], theta) * k).sum())
        assert abs(float((qm * kn).sum()) - ref) < 1e-9


def test_logical_cache_prefill_records_for_owners_only():
    """LogicalCache.prefill: output is the dense masked reference; an owner records the
    prompt's K/V under ITS OWN layer (a later decode of owner and reader sees prompt + new
    token), a reader records nothing, and a non-empty owner cache is refused."""
    rng = np.random.default_rng(21)
    S, Hq, Hkv, D, W = 19, 4, 2, 8, 5
    layout = [(FULL, 0, 0), (SLIDING, W, 1), (SLIDING, W, 1), (FULL, 0, 0)]
    lc = mo.LogicalCache(layout, Hq, Hkv, D)
    K = {0: rnd(rng, S, Hkv, D), 1: rnd(rng, S, Hkv, D)}
    V = {0: rnd(rng, S, Hkv, D), 1: rnd(rng, S, Hkv, D)}
    for layer, (kind, window, owner) in enumerate(layout):
        q = rnd(rng, S, Hq, D)
        before = {k: (v[0].shape[0]) for k, v in lc.hist.items()}
        out = lc.prefill(layer, 0, q, K[owner], V[owner])
        np.testing.assert_allclose(out, dense_reference(q, K[owner], V[owner], kind, window), rtol=0, atol=1e-12)
        if owner == layer:
            assert set(lc.hist) - set(before) == {(layer, 0)}
            np.testing.assert_array_equal(lc.hist[(layer, 0)][0], K[layer])
            np.testing.assert_array_equal(lc.hist[(layer, 0)][1], V[layer])
        else:   # a reader stores nothing
            assert {k: v[0].shape[0] for k, v in lc.hist.items()} == before
    # the recorded prompt is what a following decode step sees, for owner and reader alike
    k1, v1 = rnd(rng, 1, Hkv, D), rnd(rng, 1, Hkv, D)
    lc.append(1, 0, k1, v1)
    qd = rnd(rng, Hq, D)
    Kall, Vall = np.concatenate([K[1], k1]), np.concatenate([V[1], v1])
    qs = np.zeros((S + 1, Hq, D))
    qs[S] = qd
    ref = dense_reference(qs, Kall, Vall, SLIDING, W)[S]
    for layer in (1, 2):
        np.testing.assert_allclose(lc.decode(layer, 0, qd), ref, rtol=0, atol=1e-12)
    # the other sequence slot is untouched; a second prompt into a filled owner is refused
    assert lc.history(0, 1)[0].shape[0] == 0
    with pytest.raises(mo.OracleError) as ei:
        lc.prefill(0, 0, rnd(rng, S, Hq, D), K[0], V[0])
    assert ei.value.code == mo.ERR_UNSUPPORTED
    assert lc.history(0, 0)[0].shape[0] == S


@pytest.mark.parametrize("window,whole_tiles", [(128, True), (384, True), (1024, True), (200, False), (64, False)])
def test_a_tile_of_cached_positions_is_whole_ring_pages_iff_window_is_whole_tiles(window, whole_tiles):
    # Section 3's sliding-window cache as the ring of `window` slots (token t in slot t mod window).
    # What a kernel reading cached keys in place relies on: with 16-slot pages and a window that is
    # a multiple of 128, the stored tokens of every aligned run of 128 positions sit in
    # consecutive slots that start on a multiple of 128 (eight whole pages), for any length;
    # for other windows some run wraps inside the ring or starts off a page boundary.
    layout = [(cf.SLIDING, window, 0)]
    always = True
    for n in (1, 127, 128, 129, window - 1, window, window + 1, 3 * window + 77, 5 * window):
        if n < 1:
            continue
        ph = mo.PhysicalCache(layout, 1, 8, 1, 1, max_seq_len=8192, store_values=False)
        ph.append(0, [0], [n])
        lo = max(0, n - window)
        for t in range(lo // 128, (n - 1) // 128 + 1):
            stored = [p for p in range(128 * t, 128 * t + 128) if lo <= p < n]
            slots = [ph.locate(0, 0, p)[1] for p in stored]
            first = slots[0] - (stored[0] - 128 * t)       # slot the tile's first position would have
            ok = first % 128 == 0 and first + 128 <= window and slots == [first + (p - 128 * t) for p in stored]
            always = always and ok
    assert always == whole_tiles
