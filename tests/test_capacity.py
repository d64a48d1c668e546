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
