"""Pins for the oracle's window scorer, pooling, selection and compaction."""
import math

import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(11)


def _brute_scores(Q, K, scale):
    """Pure-Python causal attention of the window rows, summed per prefix key."""
    G, w, d = Q.shape
    N = K.shape[0]
    P = N - w
    raw = [0.0] * P
    for g in range(G):
        for i in range(w):
            pos = P + i
            logits = [scale * sum(Q[g, i, a] * K[j, a] for a in range(d)) for j in range(pos + 1)]
            m = max(logits)
            ex = [math.exp(x - m) for x in logits]
            z = sum(ex)
            for j in range(P):
                raw[j] += ex[j] / z
    return np.array(raw)


@pytest.mark.parametrize("N,w,G,d", [(24, 4, 2, 8), (64, 8, 4, 16), (9, 1, 1, 4), (12, 11, 3, 5)])
def test_scores_brute_force(N, w, G, d):
    Q = RNG.normal(size=(G, w, d))
    K = RNG.normal(size=(N, d))
    scale = 1.0 / math.sqrt(d)
    np.testing.assert_allclose(oracle.window_scores(Q, K), _brute_scores(Q, K, scale), rtol=1e-12, atol=1e-15)


@pytest.mark.parametrize("N,w,G,d", [(24, 4, 2, 8), (40, 7, 3, 16), (9, 1, 1, 4)])
def test_window_lse_against_library_logsumexp_and_the_scores(N, w, G, d):
    # pinned three ways: scipy's logsumexp of a numpy matrix product on every row's visible keys; the closed form
    # for equal keys; and the identity softmax(s)[j] = exp(s[j] - lse), which must rebuild the window scores
    from scipy.special import logsumexp
    Q = RNG.normal(size=(G, w, d)) * 3.0
    K = RNG.normal(size=(N, d))
    scale = 0.37
    P = N - w
    lse = oracle.window_lse(Q, K, scale)
    assert lse.shape == (G, w)
    rebuilt = np.zeros(P)
    for g in range(G):
        for i in range(w):
            lg = scale * (K[:P + i + 1] @ Q[g, i])
            assert abs(lse[g, i] - logsumexp(lg)) < 1e-12 * max(1.0, abs(lse[g, i]))
            rebuilt += np.exp(lg[:P] - lse[g, i])
    np.testing.assert_allclose(rebuilt, oracle.window_scores(Q, K, scale), rtol=1e-12, atol=1e-300)
    Ke = np.tile(K[:1], (N, 1))
    lse_e = oracle.window_lse(Q, Ke, scale)
    for g in range(G):
        for i in range(w):
            assert abs(lse_e[g, i] - (scale * float(Ke[0] @ Q[g, i]) + math.log(P + i + 1))) < 1e-12
    # a key the row cannot see must not enter: changing the last key only moves the last row's value
    K2 = K.copy()
    K2[N - 1] += 5.0
    d_lse = oracle.window_lse(Q, K2, scale) - lse
    assert not np.any(d_lse[:, :w - 1]) and np.abs(d_lse[:, w - 1]).min() > 0.0


def test_scores_equal_keys_closed_form():
    # all keys equal => every visible key gets 1/(number visible); raw[j] = G * sum_i 1/(N - w + i + 1)
    N, w, G, d = 40, 6, 3, 8
    K = np.tile(RNG.normal(size=(1, d)), (N, 1))
    Q = RNG.normal(size=(G, w, d))
    expect = G * sum(1.0 / (N - w + i + 1) for i in range(w))
    np.testing.assert_allclose(oracle.window_scores(Q, K), np.full(N - w, expect), rtol=1e-13)


def test_scores_single_row_is_textbook_softmax():
    from scipy.special import softmax
    N, d = 33, 8
    K = RNG.normal(size=(N, d))
    Q = RNG.normal(size=(1, 1, d))
    p = softmax(K @ Q[0, 0] / math.sqrt(d))
    np.testing.assert_allclose(oracle.window_scores(Q, K), p[:-1], rtol=1e-12)


def test_scores_mass_conservation_and_causality():
    # each row's probabilities sum to 1: prefix mass + window mass = G*w.  Window mass recomputed
    # with scipy on the window block only.
    from scipy.special import logsumexp
    N, w, G, d = 50, 5, 2, 8
    K = RNG.normal(size=(N, d))
    Q = RNG.normal(size=(G, w, d))
    raw = oracle.window_scores(Q, K)
    P = N - w
    win_mass = 0.0
    for g in range(G):
        for i in range(w):
            lg = K[:P + i + 1] @ Q[g, i] / math.sqrt(d)
            win_mass += np.exp(lg[P:] - logsumexp(lg)).sum()
    assert abs(raw.sum() + win_mass - G * w) < 1e-11
    # causality: key N-1 is visible to the last window row only, so changing it must change the
    # scores by exactly the change of that one row's contribution (a w = 1 problem on N keys)
    K2 = K.copy()
    K2[N - 1] += 3.0
    last = Q[:, w - 1:w]
    delta_last = (oracle.window_scores(last, K2) - oracle.window_scores(last, K))[:P]
    delta = oracle.window_scores(Q, K2) - raw
    assert np.abs(delta).max() > 1e-6
    np.testing.assert_allclose(delta, delta_last, rtol=0, atol=1e-14)
    # large logits do not overflow (max-subtracted)
    assert np.isfinite(oracle.window_scores(300 * Q, K)).all()


def test_pooling():
    raw = np.array([0.0, 5.0, 1.0, 2.0, 9.0, 3.0, 4.0, 0.5])
    np.testing.assert_array_equal(oracle.pool(raw, 1, 0), raw)
    np.testing.assert_array_equal(oracle.pool(raw, 3, 0), [5, 5, 5, 9, 9, 9, 4, 4])
    np.testing.assert_array_equal(oracle.pool(raw, 7, 0), [5, 9, 9, 9, 9, 9, 9, 9])
    np.testing.assert_allclose(oracle.pool(raw, 3, 1),
                               [2.5, 2.0, 8 / 3, 4.0, 14 / 3, 16 / 3, 2.5, 2.25])
    r = RNG.uniform(size=100)
    ref = [max(r[max(0, j - 3):j + 4]) for j in range(100)]
    np.testing.assert_array_equal(oracle.pool(r, 7, 0), ref)


def _brute_select(score, w, budget):
    P = len(score)
    k = budget - w
    order = sorted(range(P), key=lambda j: (-score[j], j))
    return sorted(order[:k]) + list(range(P, P + w))


@pytest.mark.parametrize("P,w,budget", [(50, 4, 14), (50, 4, 4), (50, 4, 5), (50, 4, 54), (1, 1, 2), (7, 3, 6)])
def test_select_brute_force(P, w, budget):
    s = RNG.uniform(size=P)
    s[RNG.integers(0, P, size=P // 3)] = 0.5         # many ties
    got = oracle.select(s, w, budget)
    assert got.tolist() == _brute_select(list(s), w, budget)
    assert len(got) == budget and got[-w:].tolist() == list(range(P, P + w))


def test_select_all_equal_takes_first_positions():
    got = oracle.select(np.full(30, 0.25), w=2, budget=9)
    assert got.tolist() == list(range(7)) + [30, 31]


def test_compact_is_bitwise():
    src = RNG.integers(0, 256, size=(20, 256), dtype=np.uint8)
    idx = np.array([0, 3, 4, 19, 18], dtype=np.int32)
    out = oracle.compact(src, idx)
    assert out.tobytes() == src[idx].tobytes()


# ------------------------------------------------------------------ hidden-state eviction scores
def _brute_last_token(q, K, scale):
    Hq, d = q.shape
    H, N, _ = K.shape
    G = Hq // H
    out = [0.0] * N
    for h in range(Hq):
        lg = [scale * sum(q[h, a] * K[h // G, j, a] for a in range(d)) for j in range(N)]
        m = max(lg)
        ex = [math.exp(x - m) for x in lg]
        z = sum(ex)
        for j in range(N):
            out[j] += ex[j] / z
    return np.array(out)


@pytest.mark.parametrize("H,Hq,N,d", [(2, 4, 19, 6), (1, 1, 33, 8), (3, 3, 7, 4), (2, 8, 40, 5)])
def test_last_token_scores_brute_force(H, Hq, N, d):
    q = RNG.normal(size=(Hq, d))
    K = RNG.normal(size=(H, N, d))
    np.testing.assert_allclose(oracle.last_token_scores(q, K), _brute_last_token(q, K, 1 / math.sqrt(d)),
                               rtol=1e-12, atol=1e-15)


def test_last_token_scores_closed_forms():
    from scipy.special import softmax
    # one head: a textbook softmax row; every head's probabilities sum to one => total mass Hq
    q = RNG.normal(size=(1, 8))
    K = RNG.normal(size=(1, 25, 8))
    np.testing.assert_allclose(oracle.last_token_scores(q, K), softmax(K[0] @ q[0] / math.sqrt(8)), rtol=1e-12)
    q = RNG.normal(size=(6, 8))
    K = RNG.normal(size=(2, 30, 8))
    s = oracle.last_token_scores(q, K)
    assert abs(s.sum() - 6.0) < 1e-12
    # equal keys: every position gets Hq / N
    K[:] = K[:, :1, :]
    np.testing.assert_allclose(oracle.last_token_scores(q, K), np.full(30, 6 / 30), rtol=1e-13)
    # the grouped-query mapping: head h reads KV head h // G (swap the KV heads <=> swap the query groups)
    K = RNG.normal(size=(2, 30, 8))
    a = oracle.last_token_scores(q, K)
    b = oracle.last_token_scores(np.concatenate([q[3:], q[:3]]), K[::-1])
    np.testing.assert_allclose(a, b, rtol=1e-13)
    # agreement with the window scorer's definition for a window of one row
    win = sum(oracle.window_scores(q[h * 3:(h + 1) * 3, None, :], K[h]) for h in range(2))
    np.testing.assert_allclose(a[:-1], win, rtol=1e-12)
