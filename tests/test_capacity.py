"""Cache capacity per layout (the paper's max-tokens comparison, Section 5.4) from the library's
own byte counts, against the checker's closed form and the 1/l sharing law (Section 3)."""
from oracle import mixattn_oracle as mo
from synth import configs as cf
from paper_2409_15012_b200 import build as mbuild

mbuild.build()
from paper_2409_15012_b200 import binding as mx, capacity  # noqa: E402


def test_capacity_matches_closed_form_and_sharing_law():
    Hq, Hkv, D, ctx, W = 12, 3, 128, 32000, 1024       # the paper's head counts; 32K context, s = 1024
    per_tok = 2 * Hkv * D * 2
    layouts = {
        "standard": cf.layout_all_full(24),
        "sliding": cf.layout_all_sliding(24, W),
        "mix": cf.layout_mid(W),
        "mix_pairs": cf.layout_pairs(W),
    }
    budget = 80 * 10**9
    tab = capacity.capacity_table(layouts, Hq, Hkv, D, mx.BF16, ctx, budget)
    pages = -(-ctx // 16) * 16
    assert tab["standard"][0] == 24 * pages * per_tok
    assert tab["sliding"][0] == 24 * W * per_tok
    assert tab["mix"][0] == pages * per_tok + 2 * W * per_tok
    assert tab["mix_pairs"][0] == pages * per_tok + 12 * W * per_tok
    for name, lay in layouts.items():
        ph = mo.PhysicalCache(lay, Hkv, D, 1, pages // 16, store_values=False)
        assert tab[name][0] == ph.cache_bytes(2)
        per_seq, n, total = tab[name]
        assert capacity.cache_bytes(lay, Hq, Hkv, D, mx.BF16, 3, ctx) == 3 * per_seq      # linear in sequences
        assert n == budget // per_seq and total == n * ctx
    # one shared full cache instead of 24 private ones: 1/24 of the full-attention bytes
    assert tab["standard"][0] == 24 * (tab["mix"][0] - 2 * W * per_tok)
    assert tab["mix"][1] > 20 * tab["standard"][1]


def test_named_variants_have_the_properties_the_paper_states():
    # Sections 5.1 and 5.2 fix these facts in words; the exact layer indices (figures) are parameters
    V = {k: f() for k, f in cf.PAPER_VARIANTS.items()}
    for name, lay in V.items():
        assert len(lay) == 24
        mo.validate_layout(lay)
        ctx = mx.Context(lay, 12, 3, 128, mx.BF16, 2, 8, device=-1)      # the library accepts it too
        ctx.close()
    full_owners = lambda lay: [l for l, (k, _, o) in enumerate(lay) if k == cf.FULL and o == l]
    full_layers = lambda lay: [l for l, (k, _, o) in enumerate(lay) if k == cf.FULL]
    # MA: a single standard cache, the first layer's; all other standard layers share it
    assert full_owners(V["MA"]) == [0] and len(full_layers(V["MA"])) > 2
    assert V["MA"][23][0] == cf.FULL
    # MA-EndSlide: the same, but the last layer is a sliding-window layer
    assert full_owners(V["MA-EndSlide"]) == [0] and V["MA-EndSlide"][23][0] == cf.SLIDING
    assert full_layers(V["MA-EndSlide"]) == [l for l in full_layers(V["MA"]) if l != 23]
    # MA-Offset: one standard cache, computed a few layers in, after sliding-window layers
    off = full_owners(V["MA-Offset"])
    assert len(off) == 1 and off[0] > 0 and all(V["MA-Offset"][l][0] == cf.SLIDING for l in range(off[0]))
    # MA-Pairs: two standard caches, at the first and the thirteenth layer, each shared with one more layer
    assert full_owners(V["MA-Pairs"]) == [0, 12]
    for o in (0, 12):
        assert sum(1 for l, (k, _, ow) in enumerate(V["MA-Pairs"]) if k == cf.FULL and ow == o and l != o) == 1
    # -SlideShare: strictly fewer rings than the base variant, same standard layers
    rings = lambda lay: len([l for l, (k, _, o) in enumerate(lay) if k == cf.SLIDING and o == l])
    for base in ("MA-Offset", "MA-Pairs"):
        assert rings(V[base + "-SlideShare"]) < rings(V[base])
        assert full_layers(V[base + "-SlideShare"]) == full_layers(V[base])
    # NoShare-k: k standard layers, none shared
    for k in (1, 2, 3):
        lay = V[f"MA-NoShare-{k}"]
        assert full_owners(lay) == full_layers(lay) and len(full_layers(lay)) == k
    # Successive-k (Appendix A.1): standard layers come in consecutive pairs, the second reading the
    # first's cache; the variants differ in the pairs' positions and distance, MA-Pairs-like otherwise
    seen = set()
    for k in (1, 2, 3, 4):
        lay = V[f"MA-Successive-{k}"]
        owners, layers = full_owners(lay), full_layers(lay)
        assert len(owners) == 2 and layers == sorted(owners + [o + 1 for o in owners])
        assert all(lay[o + 1] == (cf.FULL, 0, o) for o in owners)
        seen.add((owners[0], owners[1] - owners[0]))
    assert len(seen) == 4 and len({g for _, g in seen}) > 1 and len({f for f, _ in seen}) > 1
    # cache bytes: every MixAttention variant is far below the standard model at 32K tokens
    tab = capacity.capacity_table(V, 12, 3, 128, mx.BF16, 32000, 80 * 10**9)
    for name in V:
        if name.startswith("MA"):
            assert tab[name][0] * 5 < tab["standard"][0]


def test_quantised_storage_scales_every_layout_by_129_over_256():
    V = {k: f() for k, f in cf.PAPER_VARIANTS.items()}
    a = capacity.capacity_table(V, 12, 3, 128, mx.BF16, 32000, 150 * 10**9)
    b = capacity.capacity_table(V, 12, 3, 128, mx.BF16, 32000, 150 * 10**9, kv_format=mx.KV_FP8_E4M3)
    for name in V:
        assert b[name][0] * 256 == a[name][0] * 129
        assert b[name][1] >= a[name][1] * 256 // 129 - 1
