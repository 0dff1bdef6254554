"""The seeded input recipes: shapes, padding, fault structure, determinism."""
import numpy as np
import pytest
import torch

from paper_1805_10032_b200 import synthetic as syn

SMALL = {
    1: dict(),
    2: dict(dims=(48, 16, 16, 10)),
    3: dict(dims=(48, 16, 16, 10), m=20, b=8, faults=[(4, "signflip"), (4, "omniscient")]),
    4: dict(dims=(64, 32, 32, 24)),
    5: dict(d=4096),
}


@pytest.mark.parametrize("index", [1, 2, 3, 4, 5])
def test_recipe_shapes_and_padding(index):
    w = syn.make_config(index, **SMALL[index])
    assert w.V.shape == (w.m, w.ldv) and w.ldv % 32 == 0 and w.ldv >= w.d
    assert w.x.shape == (w.d,)
    assert w.features.shape == (w.n_r, w.dims[0]) and w.features.dtype == torch.float32
    assert w.d == syn.param_count(w.kind, w.dims, w.has_bias)
    if w.ldv > w.d:
        assert torch.isnan(w.V[:, w.d:].float()).all()
    assert torch.isfinite(w.V[:, :w.d].float()).all()
    assert w.V.dtype == (torch.bfloat16 if w.dtype == "bf16" else torch.float32)
    assert w.targets.dtype == (torch.float32 if w.kind == "lsq" else torch.int32)
    assert 0 <= w.b < w.m


def test_recipe_is_deterministic_and_seed_dependent():
    a = syn.make_config(2, **SMALL[2])
    b = syn.make_config(2, **SMALL[2])
    c = syn.make_config(2, seed=5, **SMALL[2])
    assert torch.equal(a.V[:, :a.d], b.V[:, :b.d]) and torch.equal(a.x, b.x)
    assert not torch.equal(a.V[:, :a.d], c.V[:, :c.d])


def test_sign_flip_rows_are_identical_copies():
    w = syn.make_config(1)
    bad = w.V[~w.honest, :w.d]
    assert bad.shape[0] == 8 and (bad == bad[0]).all()
    good = w.V[w.honest, :w.d]
    # faulty = -4 g, honest = g + noise: the honest mean is close to -faulty/4
    g = -bad[0] / 4
    assert (good.mean(0) - g).abs().mean() < 0.1


def test_config_sizes_match_the_benchmark_table():
    assert syn.param_count("mlp", (784, 10)) == 7850
    assert syn.param_count("mlp", (3072, 512, 512, 10)) == 1841162
    assert syn.param_count("mlp", (4096, 4096, 4096, 1000)) == 37659624


def test_worker_gradient_is_the_softmax_regression_gradient():
    # autograd of the generator vs the textbook closed form (p - e_y) x^T / n
    gen = torch.Generator().manual_seed(0)
    dims = (6, 3)
    x = torch.randn(syn.param_count("mlp", dims), generator=gen) * 0.2
    feats = torch.randn(5, 6, generator=gen)
    labels = torch.tensor([0, 2, 1, 1, 0], dtype=torch.int32)
    g = syn.mlp_gradient(x, dims, True, feats, labels)
    W = x[:18].view(3, 6); bvec = x[18:]
    p = torch.softmax(feats @ W.t() + bvec, dim=1)
    p[torch.arange(5), labels.long()] -= 1
    want = torch.cat([(p.t() @ feats).reshape(-1) / 5, p.mean(0)])
    assert torch.allclose(g, want, atol=1e-6)
