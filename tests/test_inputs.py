"""Seeded input generators: graph structure, gossip-matrix properties, objective data recipe."""
import numpy as np
import pytest

from paper_2006_08085_b200 import inputs


@pytest.mark.parametrize("name", list(inputs.CONFIGS))
def test_config_gossip_matrix_is_symmetric_doubly_stochastic(name):
    cfg = inputs.CONFIGS[name]
    w = inputs.gossip_matrix(cfg)
    m = w.to_dense()
    assert w.n == cfg.n
    assert np.allclose(m.sum(0), 1, atol=1e-14) and np.allclose(m.sum(1), 1, atol=1e-14)
    assert np.array_equal(m, m.T) and (m >= 0).all()
    for i in range(w.n):
        cols = w.col_idx[w.row_ptr[i]:w.row_ptr[i + 1]]
        assert (np.diff(cols) > 0).all() and i in cols
    deg = {"ring": 2, "torus8x8": 4, "regular4": 4}[cfg.graph]
    assert w.nnz == cfg.n * (deg + 1)
    assert np.allclose(w.vals, 1.0 / (deg + 1))


def test_regular4_graph_is_seeded_and_connected():
    a = inputs.random_regular4_graph(32, 4)
    assert a == inputs.random_regular4_graph(32, 4)
    assert a != inputs.random_regular4_graph(32, 5)
    seen, todo = {0}, [0]
    while todo:
        for v in a[todo.pop()]:
            if v not in seen:
                seen.add(v)
                todo.append(v)
    assert len(seen) == 32
    assert all(len(set(nb)) == 4 and i not in nb for i, nb in enumerate(a))
    assert all(i in a[j] for i, nb in enumerate(a) for j in nb)


def test_metropolis_on_irregular_graph_and_slack_and_directed():
    w = inputs.metropolis_weights(inputs.path_graph(5)).to_dense()
    assert np.allclose(w.sum(0), 1) and np.allclose(w, w.T)
    assert w[0, 1] == pytest.approx(1 / 3) and w[0, 0] == pytest.approx(2 / 3)
    s = inputs.slack_matrix(inputs.metropolis_weights(inputs.ring_graph(6)), 0.1).to_dense()
    assert s[0, 0] == pytest.approx(0.1 / 3 + 0.9) and s[0, 1] == pytest.approx(0.1 / 3)
    d = inputs.directed_cycle_blend(5).to_dense()
    assert np.allclose(d.sum(0), 1) and np.allclose(d.sum(1), 1) and not np.allclose(d, d.T)


def test_objective_data_random_access_and_types():
    cfg = inputs.CONFIGS["cfg5"].with_d(3 * inputs.BLOCK + 1234)
    lo, hi = inputs.BLOCK - 7, 2 * inputs.BLOCK + 9
    a, c, x0 = inputs.objective_data(cfg, lo, hi)
    assert a.dtype == c.dtype == x0.dtype == np.float32 and a.shape == (32, hi - lo)
    a2, c2, _ = inputs.objective_data(cfg, lo + 100, hi - 5000, threads=3)
    assert np.array_equal(a[:, 100:-5000], a2) and np.array_equal(c[:, 100:-5000], c2)
    tail = inputs.objective_data(cfg, cfg.d - 10, cfg.d)[0]
    assert tail.shape == (32, 10)


def test_objective_distributions_follow_the_configs():
    m = 60_000
    # cfg5: a ~ LogUniform[0.01, 100], c ~ N(mu_i, 1), mu_i ~ U[-5, 5], x0 = 0
    cfg = inputs.CONFIGS["cfg5"]
    a, c, x0 = inputs.objective_data(cfg, 0, m)
    la = np.log(a.astype(np.float64))
    assert a.min() >= 0.01 * (1 - 1e-6) and a.max() <= 100 * (1 + 1e-6)
    assert la.mean() == pytest.approx(0.0, abs=0.02) and la.std() == pytest.approx(np.log(1e4) / np.sqrt(12), rel=0.01)
    mu = inputs.worker_means(cfg)
    assert (np.abs(mu) <= 5).all() and np.allclose(c.mean(1), mu, atol=0.03)
    assert np.allclose(c.std(1), 1.0, atol=0.02) and not x0.any()
    # cfg1: mu_i = i - 3.5 ; a ~ U[0.5, 2]
    cfg = inputs.CONFIGS["cfg1"]
    a, c, _ = inputs.objective_data(cfg)
    assert np.allclose(inputs.worker_means(cfg), np.arange(8) - 3.5)
    assert 0.5 <= a.min() and a.max() <= 2.0 and a.mean() == pytest.approx(1.25, abs=0.01)
    # cfg2: one x0 draw per coordinate, replicated on all workers
    cfg = inputs.CONFIGS["cfg2"]
    _, _, x0 = inputs.objective_data(cfg, 0, m)
    assert (x0 == x0[0]).all() and x0[0].std() == pytest.approx(0.01, rel=0.02)
    # cfg4: mu_i = 4 sin(2 pi i / 256), c std 0.5 ; cfg3: a ~ U[0.1, 10]
    cfg = inputs.CONFIGS["cfg4"]
    assert np.allclose(inputs.worker_means(cfg), 4 * np.sin(2 * np.pi * np.arange(256) / 256))
    c = inputs.objective_data(cfg, 0, 20_000)[1]
    assert np.allclose(c.std(1), 0.5, atol=0.02)
    a = inputs.objective_data(inputs.CONFIGS["cfg3"], 0, 20_000)[0]
    assert 0.1 <= a.min() and a.max() <= 10.0
