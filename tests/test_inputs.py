"""The seeded input generators: determinism, distributions, tree shape rules."""
import math

import torch

from paper_2407_12021_b200 import inputs as gen


def test_streams_are_deterministic_and_order_free():
    a = gen.normal((1000,), 0.02, 7, 3)
    b = gen.normal((1000,), 0.02, 7, 3, chunk=128)
    assert torch.equal(a, b)
    assert not torch.equal(a, gen.normal((1000,), 0.02, 7, 4))
    assert not torch.equal(a, gen.normal((1000,), 0.02, 8, 3))
    u = gen.uniform01(100000, 1, 1)
    assert 0.0 < float(u.min()) and float(u.max()) < 1.0
    assert abs(float(u.mean()) - 0.5) < 5e-3


def test_normal_moments():
    z = gen.normal((400000,), 0.02, 5, 9, dtype=torch.float64)
    assert abs(float(z.mean())) < 2e-4
    assert abs(float(z.std()) - 0.02) < 2e-4
    assert abs(float((z / 0.02).pow(4).mean()) - 3.0) < 0.1


def test_zipf_frequencies():
    v = 1000
    t = gen.zipf_tokens(200000, v, 3, 1)
    assert int(t.min()) >= 0 and int(t.max()) < v
    h = sum(r ** -1.1 for r in range(1, v + 1))
    for r in (1, 2, 10):
        p = r ** -1.1 / h
        got = float((t == r - 1).double().mean())
        assert abs(got - p) < 4 * math.sqrt(p / 200000) + 1e-4


def test_tree_rules():
    for n, d, b, seed in ((16, 4, 4, 1), (64, 6, 4, 2), (128, 8, 6, 3), (1, 0, 1, 4), (5, 4, 2, 5)):
        tok, par = gen.make_tree(n, d, b, 32000, seed)
        assert len(tok) == len(par) == n and par[0] == -1
        dep = gen.tree_depths(par)
        assert all(0 <= par[i] < i for i in range(1, n))
        assert max(dep) == min(d, n - 1)
        for p in range(n):
            kids = [tok[i] for i in range(n) if par[i] == p]
            assert len(kids) <= max(b, 1) and len(set(kids)) == len(kids)
    assert gen.make_tree(64, 6, 4, 32000, 2) == gen.make_tree(64, 6, 4, 32000, 2)


def test_expand_tree_from_topk():
    table = {(1, 2): [3, 4], (2, 3): [5], (2, 4): [6, 7], (3, 5): [8]}
    look = lambda a, b: table.get((a, b), []) + [-1]
    tok, par, n_real = gen.expand_tree_from_topk(1, 2, look, 16, 3, 100, 0, fill=False)
    assert tok == [2, 3, 4, 5, 6, 7, 8] and par == [-1, 0, 0, 1, 2, 2, 3] and n_real == 7
    tok, par, n_real = gen.expand_tree_from_topk(1, 2, look, 16, 3, 100, 0, fill=True)
    assert len(tok) == 16 and n_real == 7 and tok[:7] == [2, 3, 4, 5, 6, 7, 8]
    assert all(0 <= par[i] < i for i in range(1, 16)) and max(gen.tree_depths(par)) <= 3
    for p in range(16):
        kids = [tok[i] for i in range(16) if par[i] == p]
        assert len(set(kids)) == len(kids)
    tok, par, n_real = gen.expand_tree_from_topk(1, 2, look, 4, 3, 100, 0)
    assert tok == [2, 3, 4, 5] and n_real == 4


def test_weight_layout_and_bytes():
    w = gen.model_weights(gen.TINY, 1)
    assert w["embed"].shape == (4096, 256) and w["layers"][1]["wgu"].shape == (1376, 256)
    assert w["layers"][0]["wqkv"].dtype == torch.float32
    assert gen.LLAMA7B.params_per_layer == 202_375_168
    assert abs(gen.LLAMA7B.weight_bytes_per_step / 1e9 - 13.21) < 0.01
    assert gen.LLAMA7B.kv_bytes_per_position() == 524288
