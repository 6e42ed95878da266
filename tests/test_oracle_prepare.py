"""Pins of the preparation-stage oracle (paper Section 3.3.1, the averaged effective rank; Algorithm 1, per-sample
grouping and majority vote): hand-worked cases, invariants, special cases that reduce to a library routine."""
import numpy as np
import pytest

import oracle


def test_mean_is_the_library_mean_and_a_worked_case():
    r = np.random.default_rng(0)
    e = r.uniform(1, 32, size=(37, 3, 5))
    np.testing.assert_allclose(oracle.prepare_mean(e), e.mean(axis=0), rtol=1e-14)
    e = np.array([[[1.0, 5.0]], [[3.0, 6.0]], [[8.0, 1.0]]])           # S = 3, L = 1, H = 2
    np.testing.assert_array_equal(oracle.prepare_mean(e), [[4.0, 4.0]])


def test_group_labels_worked_cases():
    v = np.array([[3.0, 9.0, 1.0, 7.0, 5.0, 2.0]])
    # descending: 9 7 5 3 2 1 -> heads 1 3 4 0 5 2; M = 3: two heads per group
    np.testing.assert_array_equal(oracle.group_labels(v, 3), [[1, 0, 2, 0, 1, 2]])
    # M = 4 with n = 6: floor boundaries 0, 1, 3, 4, 6 -> sizes 1, 2, 1, 2
    np.testing.assert_array_equal(oracle.group_labels(v, 4), [[2, 0, 3, 1, 1, 3]])
    # M = n: the label is the rank;  M = 1: one group
    np.testing.assert_array_equal(oracle.group_labels(v, 6), [[3, 0, 5, 1, 2, 4]])
    np.testing.assert_array_equal(oracle.group_labels(v, 1), np.zeros((1, 6), dtype=np.int32))
    # equal values: the lower index ranks first
    np.testing.assert_array_equal(oracle.group_labels(np.array([[2.0, 2.0, 2.0, 2.0]]), 2), [[0, 0, 1, 1]])
    with pytest.raises(ValueError):
        oracle.group_labels(v, 7)


def test_group_labels_against_argsort_and_scopes():
    r = np.random.default_rng(1)
    v = r.permutation(24).astype(np.float64).reshape(4, 6)
    for M in (2, 3, 6):
        per_layer = oracle.group_labels(v, M)
        for l in range(4):
            rank = np.empty(6, dtype=int)
            rank[np.argsort(-v[l], kind="stable")] = np.arange(6)
            np.testing.assert_array_equal(per_layer[l], rank * M // 6)      # n divisible by M: floor(r M / n)
    whole = oracle.group_labels(v, 4, scope=1)
    rank = np.empty(24, dtype=int)
    rank[np.argsort(-v.ravel(), kind="stable")] = np.arange(24)
    np.testing.assert_array_equal(whole.ravel(), rank * 4 // 24)
    # sizes differ by at most one and the groups are ordered by value
    v = r.standard_normal((1, 11))
    lab = oracle.group_labels(v, 4)[0]
    sizes = np.bincount(lab, minlength=4)
    assert sizes.sum() == 11 and sizes.max() - sizes.min() <= 1
    for g in range(3):
        assert v[0][lab == g].min() > v[0][lab == g + 1].max()


def test_majority_vote_worked_case_and_ties():
    # L = 1, H = 2, M = 2: head with the larger value gets label 0
    e = np.array([[[5.0, 1.0]], [[4.0, 2.0]], [[1.0, 9.0]]])
    votes, lab = oracle.majority_vote(e, 2)
    np.testing.assert_array_equal(votes, [[[2, 1], [1, 2]]])
    np.testing.assert_array_equal(lab, [[0, 1]])
    # a tie between groups goes to the lower group
    votes, lab = oracle.majority_vote(e[[0, 2]], 2)
    np.testing.assert_array_equal(votes, [[[1, 1], [1, 1]]])
    np.testing.assert_array_equal(lab, [[0, 0]])


def test_majority_vote_invariants():
    r = np.random.default_rng(2)
    base = r.uniform(1, 32, size=(4, 8))
    # identical samples: the vote is unanimous and equals the labels of the mean
    e = np.repeat(base[None], 9, axis=0)
    votes, lab = oracle.majority_vote(e, 4)
    np.testing.assert_array_equal(lab, oracle.group_labels(oracle.prepare_mean(e), 4))
    assert (votes.max(axis=2) == 9).all() and (votes.sum(axis=2) == 9).all()
    # noisy samples: votes add up to S per head; per sample and group the head counts are the group sizes
    e = base[None] + r.standard_normal((51, 4, 8))
    for scope in (0, 1):
        votes, lab = oracle.majority_vote(e, 4, scope)
        assert (votes.sum(axis=2) == 51).all()
        n_sets = 4 if scope == 0 else 1
        assert (votes.sum(axis=(0, 1)) == 51 * 32 // 4).all() and votes.reshape(n_sets, -1, 4).sum(axis=1).max() == 51 * 32 // 4 // n_sets
        np.testing.assert_array_equal(lab, votes.argmax(axis=2))       # argmax takes the first maximum
        # the order of the samples does not matter
        v2, l2 = oracle.majority_vote(e[::-1], 4, scope)
        np.testing.assert_array_equal(v2, votes)


def test_retrieval_layer_worked_cases():
    # layer means 4, 3, 5, 5.5, 2: rises of -1, +2, +0.5, -3.5 -> the layer after the +2 rise is layer 2
    v = np.array([[4.0, 4.0], [2.0, 4.0], [6.0, 4.0], [5.0, 6.0], [1.0, 3.0]])
    layer, inc = oracle.retrieval_layer(v)
    assert layer == 2
    np.testing.assert_allclose(inc, [-1.0, 2.0, 0.5, -3.5], rtol=1e-15)
    # equal rises: the earliest layer;  monotone decrease: the smallest drop wins;  two layers: layer 1
    assert oracle.retrieval_layer(np.array([[0.0], [1.0], [2.0], [3.0]]))[0] == 1
    assert oracle.retrieval_layer(np.array([[9.0], [5.0], [4.5], [1.0]]))[0] == 2
    assert oracle.retrieval_layer(np.array([[3.0, 1.0], [0.0, 0.0]]))[0] == 1
    # against numpy on random values
    r = np.random.default_rng(4)
    for _ in range(50):
        v = r.standard_normal((int(r.integers(2, 40)), int(r.integers(1, 9))))
        layer, inc = oracle.retrieval_layer(v)
        m = v.mean(axis=1)
        np.testing.assert_allclose(inc, np.diff(m), rtol=1e-12, atol=1e-15)
        assert layer == int(np.argmax(inc)) + 1
