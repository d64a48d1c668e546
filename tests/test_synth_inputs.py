"""The seeded generators: deterministic, chunk-independent, roughly N(0,1)."""
import numpy as np
import torch

from synth import inputs as si
from synth import configs as cf


def test_values_do_not_depend_on_chunking():
    K, V = si.kv_tokens(1, 0, 3, 0, 40, 2, 16, torch.float32)
    K2, V2 = si.kv_tokens(1, 0, 3, 17, 5, 2, 16, torch.float32)
    assert torch.equal(K[17:22], K2) and torch.equal(V[17:22], V2)
    q = si.q_tokens(1, 2, 3, 0, 9, 4, 16, torch.bfloat16)
    assert torch.equal(q[8:9], si.q_tokens(1, 2, 3, 8, 1, 4, 16, torch.bfloat16))


def test_streams_differ_and_moments():
    K, V = si.kv_tokens(5, 1, 0, 0, 4096, 2, 64, torch.float32)
    K2, _ = si.kv_tokens(5, 1, 1, 0, 4096, 2, 64, torch.float32)
    K3, _ = si.kv_tokens(6, 1, 0, 0, 4096, 2, 64, torch.float32)
    assert not torch.equal(K, V) and not torch.equal(K, K2) and not torch.equal(K, K3)
    x = K.double().numpy().ravel()
    assert abs(x.mean()) < 0.01 and abs(x.var() - 1.0) < 0.01
    assert abs(np.corrcoef(x[:-1], x[1:])[0, 1]) < 0.01
    assert 3.5 < np.abs(x).max() < 4.9


def test_large_counter_uses_high_bits():
    a = si.unit_normal(123, torch.tensor([5, 5 + (1 << 32), 5 + (2 << 32)]))
    assert len(set(a.tolist())) == 3


def test_lengths_and_permutation():
    n = si.draw_lengths(4, 64, 1024, 65536)
    assert n.min() >= 1024 and n.max() <= 65536 and len(n) == 64
    assert np.array_equal(n, si.draw_lengths(4, 64, 1024, 65536))
    p = si.page_permutation(4, 1000)
    assert sorted(p.tolist()) == list(range(1000)) and p.tolist() != list(range(1000))


def test_layouts():
    mid = cf.layout_mid(1024)
    assert len(mid) == 24 and cf.owners_of(mid) == [0, 1, 13]
    assert mid[12] == (cf.FULL, 0, 0) and mid[11] == (cf.SLIDING, 1024, 1) and mid[23][2] == 13
    pairs = cf.layout_pairs(1024)
    assert pairs[2][2] == 1 and pairs[11][2] == 11 and pairs[13][2] == 13 and pairs[14][2] == 13
    assert pairs[23][2] == 23 and pairs[12] == (cf.FULL, 0, 0)


def test_multi_and_head_variants_agree():
    K, V = si.kv_tokens(3, 1, 4, 10, 6, 2, 16, torch.bfloat16)
    Km, Vm = si.kv_tokens_multi(3, 1, [2, 4], [0, 10], 6, 2, 16, torch.bfloat16)
    assert torch.equal(Km[1], K) and torch.equal(Vm[1], V)
    assert torch.equal(Km[0], si.kv_tokens(3, 1, 2, 0, 6, 2, 16, torch.bfloat16)[0])
    Kh, Vh = si.kv_tokens_head(3, 1, 4, 10, 6, 2, 16, 1, torch.bfloat16)
    assert torch.equal(Kh, K[:, 1]) and torch.equal(Vh, V[:, 1])
    qm = si.q_tokens_multi(3, 2, [2, 4], [5, 10], 3, 4, 16, torch.bfloat16)
    assert torch.equal(qm[1], si.q_tokens(3, 2, 4, 10, 3, 4, 16, torch.bfloat16))
    assert torch.equal(qm[0], si.q_tokens(3, 2, 2, 5, 3, 4, 16, torch.bfloat16))
