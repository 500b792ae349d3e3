"""Pins for the oracle's shuffled sample order (Algorithm 1 read literally: shuffle the shard once, then take
the n-th example, cycling when a node runs longer than its shard). What the mathematics fixes: the first m draws
are a permutation of the shard, the order repeats with period m, nodes and seeds get different orders, and every
row is equally likely at any given position. Not GPU."""
import numpy as np
import pytest

import oracle


@pytest.fixture(autouse=True)
def shuffled_mode():
    oracle.set_sampling(1)
    yield
    oracle.set_sampling(0)


@pytest.mark.parametrize("m", [1, 2, 3, 4, 5, 7, 8, 9, 63, 64, 65, 1000, 4096, 4097, 65537])
def test_one_cycle_is_a_permutation_and_repeats(m):
    a = oracle.sample_indices(11, 2, m, 0, 2 * m + 5)
    assert np.array_equal(np.sort(a[:m]), np.arange(m))
    assert np.array_equal(a[m:2 * m], a[:m])
    assert np.array_equal(a[2 * m:], a[:5] if m >= 5 else np.resize(a[:m], 5))


def test_chunking_independent_and_keyed_by_node_and_seed():
    m = 1000
    a = oracle.sample_indices(7, 3, m, 0, 2500)
    b = np.concatenate([oracle.sample_indices(7, 3, m, 0, 999), oracle.sample_indices(7, 3, m, 999, 2),
                        oracle.sample_indices(7, 3, m, 1001, 1499)])
    assert np.array_equal(a, b)
    assert not np.array_equal(a[:m], oracle.sample_indices(7, 4, m, 0, m))
    assert not np.array_equal(a[:m], oracle.sample_indices(8, 3, m, 0, m))
    assert not np.array_equal(a[:m], np.arange(m))


def test_positions_are_uniform_over_seeds():
    m, trials = 16, 8000
    first = np.array([oracle.sample_indices(s, 0, m, 0, 2) for s in range(trials)])
    for pos in (0, 1):
        counts = np.bincount(first[:, pos], minlength=m).astype(float)
        chi2 = ((counts - trials / m) ** 2 / (trials / m)).sum()
        assert chi2 < 60.0  # 15 degrees of freedom: mean 15, sd 5.5
    # consecutive positions are distinct rows (a permutation), and not simply neighbours
    assert (first[:, 0] != first[:, 1]).all()
    assert np.mean(np.abs(first[:, 0].astype(int) - first[:, 1].astype(int)) == 1) < 0.3


def test_one_epoch_visits_every_row_exactly_once():
    # rows = unit vectors, squared loss, no regulariser, w0 = 0, targets 1: a visit of row i sets w_i = eta and
    # touches nothing else, so after exactly one epoch w = eta * ones; with repeated or missing rows it is not
    m = d = 37
    X = np.eye(m, dtype=np.float32)
    y = np.ones(m, dtype=np.float32)
    eta = float(np.float32(0.25))
    W = oracle.run_dense(X, y, np.array([0, m]), np.array([m]), d, eta, 0, 0.0, 2, 5)
    np.testing.assert_array_equal(W[0], np.full(d, eta))
    oracle.set_sampling(0)
    W0 = oracle.run_dense(X, y, np.array([0, m]), np.array([m]), d, eta, 0, 0.0, 2, 5)
    assert not np.array_equal(W0[0], np.full(d, eta))  # independent draws repeat and miss rows
