"""The synthetic input recipes: determinism, distinct coordinates, stated size laws."""
import numpy as np
import pytest

from workloads import configs, rng


def _keys(w):
    key = np.zeros(w.nnz, dtype=np.int64)
    for d in range(w.coords.shape[1]):
        key = key * w.dims[d] + w.coords[:, d]
    return key


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_mini_workloads_are_valid_and_deterministic(cfg):
    w = configs.make(cfg, "mini")
    assert w.coords.dtype == np.int32 and w.vals.dtype == np.float32
    assert np.unique(_keys(w)).size == w.nnz
    assert (w.coords >= 0).all() and (w.coords.max(axis=0) < np.array(w.dims)).all()
    w2 = configs.make(cfg, "mini")
    assert np.array_equal(w.coords, w2.coords) and np.array_equal(w.vals, w2.vals)
    assert all(np.array_equal(a, b) for a, b in zip(w.dense, w2.dense))
    # not sorted: the builder has to sort
    assert (np.diff(_keys(w)) < 0).any()


def test_zipf_sizes_law():
    n = configs.zipf_sizes(50_000_000, 100_000, 1.2)
    assert n.sum() == 50_000_000 and n[0] == n.max()
    assert abs(n[0] / 50e6 - 0.196) < 0.002          # head slice holds ~19.6 % of the nonzeros
    assert 8 <= n[-1] <= 11
    assert np.all(np.diff(n) <= 0)


def test_powerlaw_degrees_law():
    d = configs.powerlaw_degrees(30_000_000, 1_000_000, 1.5, 50_000)
    assert d.sum() == 30_000_000 and d.max() == 50_000
    assert 150 <= (d == 50_000).sum() <= 260


def test_split_totals_exact_and_capped():
    totals = np.array([10, 0, 1, 57, 12])
    parts = np.array([3, 0, 1, 5, 12])
    s = configs.split_totals(7, 1, totals, parts, cap=30)
    assert s.min() >= 1 and s.max() <= 30
    assert np.array_equal(np.add.reduceat(s, [0, 3, 4, 9]), [10, 1, 57, 12])


def test_keyed_bijection_is_a_bijection():
    for n in (1, 2, 7, 1000, 4097):
        img = rng.keyed_bijection(np.arange(n), n, np.uint64(12345))
        assert np.array_equal(np.sort(img), np.arange(n))
    a = rng.keyed_bijection(np.arange(1000), 1000, np.uint64(1))
    b = rng.keyed_bijection(np.arange(1000), 1000, np.uint64(2))
    assert not np.array_equal(a, b)


def test_value_distributions():
    u = rng.uniform_f32(1, 1, np.arange(200000), -1.0, 1.0)
    assert u.min() >= -1 and u.max() < 1 and abs(u.mean()) < 0.01 and abs(u.var() - 1 / 3) < 0.01
    g = rng.normal_f32(1, 2, np.arange(200000))
    assert abs(g.mean()) < 0.01 and abs(g.std() - 1) < 0.01
