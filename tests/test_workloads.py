"""The synthetic input generators: shapes, padding, determinism, and the
distribution parameters of the five workload recipes (they carry no aggregation
arithmetic, so there is no oracle to compare with -- only the recipe)."""

import numpy as np
import pytest
import torch

from paper_2501_17392_b200 import workloads as W


def test_table_of_workloads():
    got = {k: (w.n, w.f, w.d, w.rounds, w.lam) for k, w in W.WORKLOADS.items()}
    assert got == {"cfg1": (8, 1, 100_000, 1, 0.0), "cfg2": (20, 4, 1_663_370, 1, 1.0),
                   "cfg3": (50, 10, 11_689_512, 1, 2.0), "cfg4": (100, 20, 25_557_032, 1, 5.0),
                   "cfg5": (16, 3, 124_439_808, 5, 0.0)}
    for w in W.WORKLOADS.values():
        assert w.ld % 128 == 0 and 0 <= w.ld - w.d < 128


@pytest.mark.parametrize("name", sorted(W.WORKLOADS))
def test_shapes_padding_and_determinism(name):
    w = W.scaled(W.WORKLOADS[name], 50_001)
    a = W.honest_updates(w, 0)
    b = W.honest_updates(w, 0)
    c = W.honest_updates(w, 1)
    assert a.shape == (w.n, w.ld) and a.dtype == torch.float32
    assert torch.equal(a, b) and not torch.equal(a, c)
    assert (a[:, w.d:] == 0).all()
    assert torch.isfinite(a).all()
    noise, unif = W.attack_draws(w, 0)
    if w.attack in (W.ATTACK_GAUSSIAN, W.ATTACK_SPARSE_NOISE):
        assert noise.shape == (w.f, w.ld) and abs(float(noise[:, :w.d].std()) - 1.0) < 0.02
    else:
        assert noise is None
    if w.attack == W.ATTACK_SPARSE_NOISE:
        u = unif[:, :w.d]
        assert float(u.min()) >= 0.0 and float(u.max()) < 1.0 and abs(float(u.mean()) - 0.5) < 0.01
        assert (unif[:, w.d:] == 1.0).all()                 # padding can never pass `u < prob`
    else:
        assert unif is None


def test_recipe_statistics():
    d = 200_000
    x = W.honest_updates(W.scaled(W.WORKLOADS["cfg1"], d)).numpy()[:, :d]
    assert abs(x.mean() - 0.01) < 1e-3 and abs(x.std() - 0.1) < 1e-3
    x = W.honest_updates(W.scaled(W.WORKLOADS["cfg2"], d)).numpy()[:, :d]
    mu = x.mean(0)
    assert abs(mu.std() - np.sqrt(0.05 ** 2 + 0.02 ** 2 / 20)) < 2e-3      # shared mean dominates
    assert abs((x - mu).std() - 0.02 * np.sqrt(19 / 20)) < 1e-3
    x = W.honest_updates(W.scaled(W.WORKLOADS["cfg3"], d)).numpy()[:, :d]
    s = x.std(1) / 0.01
    assert s.min() > 0.45 and s.max() < 2.1 and s.max() / s.min() > 1.5   # per-client heterogeneity
    x = W.honest_updates(W.scaled(W.WORKLOADS["cfg4"], d)).numpy()[:, :d]
    assert abs(x.std() - 0.01) < 1e-4
    x = W.honest_updates(W.scaled(W.WORKLOADS["cfg5"], d)).numpy()[:, :d] / 0.001
    kurt = ((x - x.mean()) ** 4).mean() / x.var() ** 2
    assert kurt > 3.05                                                     # 1% Student-t(3) entries fatten the tails
    assert abs(np.median(np.abs(x)) - 0.6745) < 0.01


def test_edge_and_integer_generators():
    x = W.edge_value_updates(5, 3000, seed=1, ld=3008)
    v = x[:, :3000]
    assert torch.isnan(v).any() and torch.isinf(v).any() and (v == 0).any()
    y = W.small_integer_updates(4, 100, seed=2)
    assert set(y.unique().tolist()) <= set(float(i) for i in range(-3, 4))
