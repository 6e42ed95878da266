"""Pins of the decode-step oracle (paper Section 3.3.3, last sentence of "Dynamic KV Cache Eviction";
Algorithm 2, decoding loop): closed forms, a library softmax, brute force on tiny inputs, invariants."""
import math

import numpy as np
import pytest
from scipy.special import softmax

import oracle


def _rand(seed, G, n, d):
    r = np.random.default_rng(seed)
    return r.standard_normal((G, d)), r.standard_normal((n, d)), r.standard_normal(d)


def test_zero_query_gives_uniform_attention():
    _, Kc, kn = _rand(0, 3, 17, 8)
    p = oracle.decode_probs(np.zeros((3, 8)), Kc, kn)
    np.testing.assert_allclose(p, np.full(18, 3.0 / 18.0), rtol=1e-14)


def test_one_hot_keys_closed_form():
    # keys a_j e_j, query e_2: only entry 2 has a non-zero logit, scale * a_2
    d, n = 16, 9
    a = np.arange(1.0, n + 1.0)
    Kc = np.zeros((n, d))
    Kc[np.arange(n), np.arange(n)] = a
    kn = np.zeros(d)
    kn[n] = 5.0
    q = np.zeros((1, d))
    q[0, 2] = 2.0
    s = 0.25 * 2.0 * a[2]            # scale 1/sqrt(16)
    p = oracle.decode_probs(q, Kc, kn)
    want = np.full(n + 1, 1.0 / (math.exp(s) + n))
    want[2] = math.exp(s) / (math.exp(s) + n)
    np.testing.assert_allclose(p, want, rtol=1e-13)
    # the new token is entry n: a query along its axis singles it out
    q[0] = 0.0
    q[0, n] = 1.0
    p = oracle.decode_probs(q, Kc, kn, scale=1.0)
    assert p.argmax() == n and abs(p[n] - math.exp(5.0) / (math.exp(5.0) + n)) < 1e-13


@pytest.mark.parametrize("G,n,d,scale", [(1, 1, 4, None), (4, 33, 128, None), (2, 7, 5, 0.3)])
def test_against_library_softmax(G, n, d, scale):
    q, Kc, kn = _rand(G * 100 + n, G, n, d)
    sc = 1.0 / math.sqrt(d) if scale is None else scale
    logits = sc * q @ np.vstack([Kc, kn]).T            # [G, n + 1]
    want = softmax(logits, axis=1).sum(axis=0)
    np.testing.assert_allclose(oracle.decode_probs(q, Kc, kn, scale), want, rtol=1e-12)
    assert abs(want.sum() - G) < 1e-12


def test_brute_force_tiny_and_head_order():
    q, Kc, kn = _rand(5, 2, 3, 2)
    rows = [list(map(float, r)) for r in Kc] + [list(map(float, kn))]
    p = [0.0] * 4
    for g in range(2):
        s = [sum(q[g][a] * r[a] for a in range(2)) / math.sqrt(2.0) for r in rows]
        z = sum(math.exp(x) for x in s)
        for j in range(4):
            p[j] += math.exp(s[j]) / z
    np.testing.assert_allclose(oracle.decode_probs(q, Kc, kn), p, rtol=1e-13)
    # summing over heads: the order of the heads does not matter, a single head differs
    np.testing.assert_allclose(oracle.decode_probs(q[::-1], Kc, kn), p, rtol=1e-13)
    assert not np.allclose(oracle.decode_probs(q[:1], Kc, kn), p)


def test_same_numbers_as_the_last_token_scorer():
    # the hidden-state eviction scorer with one KV head is the same attention, written separately
    q, Kc, kn = _rand(9, 4, 40, 16)
    np.testing.assert_allclose(oracle.decode_probs(q, Kc, kn),
                               oracle.last_token_scores(q, np.vstack([Kc, kn])[None]), rtol=1e-13)


def test_shift_of_keys_orthogonal_to_queries_changes_nothing():
    q, Kc, kn = _rand(11, 2, 12, 6)
    q[:, 5] = 0.0
    shift = np.zeros(6)
    shift[5] = 37.0
    np.testing.assert_allclose(oracle.decode_probs(q, Kc + shift, kn + shift), oracle.decode_probs(q, Kc, kn), rtol=1e-12)


def _brute_evict(cum, pos, new_pos, protect):
    cand = [j for j in range(len(cum)) if pos[j] <= new_pos - protect] or list(range(len(cum)))
    return min(cand, key=lambda j: (cum[j], pos[j]))


def test_evict_rule():
    r = np.random.default_rng(3)
    for trial in range(200):
        n = int(r.integers(1, 12))
        pos = np.sort(r.choice(40, size=n, replace=False)).astype(np.int32)
        cum = r.integers(0, 4, size=n).astype(np.float64)     # many ties
        perm = r.permutation(n)                                # the cache need not be ordered by position
        pos, cum = pos[perm], cum[perm]
        new_pos = 40
        protect = int(r.integers(1, 30))
        assert oracle.decode_evict(cum, pos, new_pos, protect) == _brute_evict(cum, pos, new_pos, protect)
    # equal scores: the older entry leaves;  protected entries stay even with the lowest score
    assert oracle.decode_evict([1.0, 1.0, 1.0], [7, 3, 5], 10, 1) == 1
    assert oracle.decode_evict([5.0, 0.0, 4.0], [1, 9, 2], 10, 2) == 2
    # nothing old enough: every cached entry is a candidate
    assert oracle.decode_evict([5.0, 0.5, 4.0], [8, 9, 7], 10, 8) == 1


def test_update_appends_below_budget_and_evicts_at_budget():
    q, Kc, kn = _rand(21, 2, 6, 8)
    Vc = np.arange(48.0).reshape(6, 8)
    vn = -np.ones(8)
    pos = np.array([0, 2, 3, 7, 8, 9], dtype=np.int32)
    cum = np.array([3.0, 0.01, 2.0, 0.5, 0.7, 0.9])
    K2, V2, pos2, cum2, p, ev = oracle.decode_update(q, Kc, Vc, pos, cum, kn, vn, new_pos=10, cap=8)
    assert ev == -1 and len(pos2) == 7 and pos2[-1] == 10 and (V2[-1] == vn).all() and (K2[:6] == Kc).all()
    np.testing.assert_allclose(cum2[:6], cum + p[:6], rtol=1e-15)
    assert cum2[6] == p[6]
    K3, V3, pos3, cum3, p3, ev3 = oracle.decode_update(q, Kc, Vc, pos, cum, kn, vn, new_pos=10, cap=6)
    assert ev3 == 2 and list(pos3) == [0, 3, 7, 8, 9, 10] and len(cum3) == 6      # entry with cum 0.01 + p < rest
    assert (K3[-1] == kn).all() and (V3[:5] == Vc[[0, 2, 3, 4, 5]]).all()
    np.testing.assert_allclose(cum3[:5], (cum + p3[:6])[[0, 2, 3, 4, 5]], rtol=1e-15)


def test_seed_of_the_cumulative_scores():
    score = np.array([0.5, 0.1, 0.9, 0.3, 0.7])                 # P = 5
    np.testing.assert_array_equal(oracle.decode_seed(score, [1, 3, 5, 6]), [0.1, 0.3, 0.3, 0.3])
    np.testing.assert_array_equal(oracle.decode_seed(score, [2, 4, 5]), [0.9, 0.7, 0.9])
    np.testing.assert_array_equal(oracle.decode_seed(score, [5, 6]), [0.0, 0.0])          # only the window is kept
    np.testing.assert_array_equal(oracle.decode_seed(-score, [0, 1, 7]), [-0.5, -0.1, -0.1])   # negative scores: still the largest
    # kept positions need not be sorted
    np.testing.assert_array_equal(oracle.decode_seed(score, [6, 0, 2]), [0.9, 0.5, 0.9])
