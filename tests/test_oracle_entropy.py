"""Pins for the oracle's covariance / eigenvalue / truncated-entropy stage (no GPU).

Each test checks the oracle against something the paper or the mathematics fixes, never against
the oracle's own formula retyped."""
import math

import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(20241003)


# ---------------------------------------------------------------------------------- covariance
def test_covariance_matches_definition_by_brute_force():
    # Eq. 1 written as explicit Python loops on a tiny input with N != d (catches a transposed
    # operand, a dropped mean, a wrong index).
    N, d = 5, 3
    X = RNG.normal(size=(N, d))
    mean = [sum(X[i][a] for i in range(N)) / N for a in range(d)]
    ref = [[sum((X[i][a] - mean[a]) * (X[i][c] - mean[c]) for i in range(N)) for c in range(d)]
           for a in range(d)]
    got = oracle.covariance(X, center=True)
    assert got.shape == (d, d)
    np.testing.assert_allclose(got, np.array(ref), rtol=1e-13, atol=1e-13)
    ref_u = [[sum(X[i][a] * X[i][c] for i in range(N)) for c in range(d)] for a in range(d)]
    np.testing.assert_allclose(oracle.covariance(X, center=False), np.array(ref_u), rtol=1e-13, atol=1e-13)


def test_covariance_matches_library_routine():
    X = RNG.normal(size=(200, 16)) + 3.0
    np.testing.assert_allclose(oracle.covariance(X) / (200 - 1), np.cov(X, rowvar=False), rtol=1e-11, atol=1e-12)


def test_covariance_rank_bounded_by_token_count():
    # Lemma 3: rank(Sigma) <= rank(X); with N < D the covariance is rank deficient.
    X = RNG.normal(size=(6, 16))
    lam = oracle.eigenvalues(oracle.covariance(X))
    assert (lam[5:] < 1e-10 * lam[0]).all()       # centring removes one more direction: rank <= N - 1
    assert lam[4] > 1e-6 * lam[0]


# --------------------------------------------------------------------------------- eigenvalues
def test_eigenvalues_2x2_closed_form():
    for a, b, c in [(2.0, 1.0, 3.0), (5.0, -2.0, 1.0), (1.0, 0.0, 4.0), (1.0, 1e-9, 1.0)]:
        mid, rad = 0.5 * (a + c), math.hypot(0.5 * (a - c), b)
        lam = oracle.eigenvalues(np.array([[a, b], [b, c]]))
        np.testing.assert_allclose(lam, [mid + rad, mid - rad], rtol=1e-13, atol=1e-15)


def test_eigenvalues_3x3_closed_form():
    # trigonometric solution of the characteristic cubic of a symmetric 3x3 matrix
    A = np.array([[4.0, 1.0, -2.0], [1.0, 2.0, 0.5], [-2.0, 0.5, 3.0]])
    q = np.trace(A) / 3.0
    p2 = ((A - q * np.eye(3)) ** 2).sum() / 6.0
    p = math.sqrt(p2)
    Bm = (A - q * np.eye(3)) / p
    r = np.linalg.det(Bm) / 2.0
    phi = math.acos(max(-1.0, min(1.0, r))) / 3.0
    e1 = q + 2 * p * math.cos(phi)
    e3 = q + 2 * p * math.cos(phi + 2 * math.pi / 3)
    e2 = 3 * q - e1 - e3
    np.testing.assert_allclose(oracle.eigenvalues(A), [e1, e2, e3], rtol=1e-12)


def _orthogonal(d, reflections=5):
    Q = np.eye(d)
    for _ in range(reflections):
        v = RNG.normal(size=d)
        v /= np.linalg.norm(v)
        Q = Q @ (np.eye(d) - 2.0 * np.outer(v, v))
    return Q


@pytest.mark.parametrize("d", [4, 17, 128])
def test_eigenvalues_of_constructed_spectrum(d):
    lam = np.sort(RNG.uniform(0.0, 10.0, size=d))[::-1]
    lam[-1] = 0.0
    if d > 4:
        lam[3] = lam[2]            # a repeated eigenvalue
    Q = _orthogonal(d)
    A = (Q * lam) @ Q.T
    A = 0.5 * (A + A.T)
    np.testing.assert_allclose(oracle.eigenvalues(A), lam, rtol=0, atol=1e-12 * lam[0])


def test_eigenvalues_trace_frobenius_and_diagonal():
    M = RNG.normal(size=(40, 40))
    A = M + M.T
    lam = oracle.eigenvalues(A)
    assert abs(lam.sum() - np.trace(A)) < 1e-11 * np.abs(A).sum()
    assert abs((lam ** 2).sum() - (A ** 2).sum()) < 1e-11 * (A ** 2).sum()
    assert (np.diff(lam) <= 0).all()
    dg = np.array([3.0, -1.0, 7.0, 0.0])
    np.testing.assert_array_equal(oracle.eigenvalues(np.diag(dg)), np.sort(dg)[::-1])
    # block diagonal: union of the blocks' spectra
    Bk = np.zeros((4, 4))
    Bk[:2, :2] = [[2, 1], [1, 2]]
    Bk[2:, 2:] = [[5, 2], [2, 5]]
    np.testing.assert_allclose(oracle.eigenvalues(Bk), [7, 3, 3, 1], atol=1e-13)


def test_eigenvalues_agree_with_lapack_on_key_matrices():
    # a library routine the oracle does not use, at the real size d = 128, on ill-conditioned input
    import torch
    from paper_2410_03090_b200 import synth
    wl = synth.WORKLOADS["c1"]
    for h in (0, 3, 7):
        K, _, _ = synth.generate_unit(wl, 0, 0, h)
        Cm = oracle.covariance(K.double().numpy())
        ref = torch.linalg.eigvalsh(torch.from_numpy(Cm)).numpy()[::-1]
        np.testing.assert_allclose(oracle.eigenvalues(Cm), ref, rtol=0, atol=1e-12 * ref[0])


# ------------------------------------------------------------------------------------- entropy
def test_entropy_rank_one_is_zero():
    # Appendix, proof of Lemma 4: H(1, 0, ..., 0) = 0, erank = 1.  Centred rank-1 data.
    u = RNG.normal(size=(64, 1))
    v = RNG.normal(size=(1, 16))
    H, E = oracle.entropy(u @ v, k_trunc=8)
    assert abs(H) < 1e-9 and abs(E - 1.0) < 1e-9
    H, E = oracle.truncated_entropy(np.array([1.0, 0, 0, 0]), k=4)
    assert H == 0.0 and E == 1.0


@pytest.mark.parametrize("m", [1, 2, 5, 8])
def test_entropy_of_m_equal_directions_is_log_m(m):
    # rows +a e_i and -a e_i for i < m: mean zero, m equal non-zero eigenvalues => erank = m = rank
    d, a = 12, 1.7
    rows = []
    for i in range(m):
        e = np.zeros(d)
        e[i] = a
        rows += [e, -e]
    H, E = oracle.entropy(np.array(rows), k_trunc=8)
    assert abs(H - math.log(m)) < 1e-12
    assert abs(E - m) < 1e-10


def test_entropy_isotropic_truncated_at_k():
    # uniform spectrum on D values: full entropy ln D (Appendix); truncated at k and renormalised
    # over the leading block: ln k; with the whole trace normalised: (k/D) ln D.
    D, k = 128, 32
    lam = np.full(D, 0.37)
    H, E = oracle.truncated_entropy(lam, k=k, norm=0)
    assert abs(H - math.log(k)) < 1e-12 and abs(E - k) < 1e-9
    H1, _ = oracle.truncated_entropy(lam, k=k, norm=1)
    assert abs(H1 - (k / D) * math.log(D)) < 1e-12
    Hf, Ef = oracle.truncated_entropy(lam, k=D, norm=1)
    assert abs(Hf - math.log(D)) < 1e-12 and abs(Ef - D) < 1e-9


def test_entropy_worked_spectrum():
    # hand-computed: spectrum (4, 2, 1, 1), k = 2 -> p = (2/3, 1/3); k = 4, trace-normalised -> p = (.5,.25,.125,.125)
    lam = np.array([4.0, 2.0, 1.0, 1.0])
    H, _ = oracle.truncated_entropy(lam, k=2, norm=0)
    assert abs(H - (-(2 / 3) * math.log(2 / 3) - (1 / 3) * math.log(1 / 3))) < 1e-14
    H, _ = oracle.truncated_entropy(lam, k=2, norm=1)
    assert abs(H - (0.5 * math.log(2) + 0.25 * math.log(4))) < 1e-14
    H, E = oracle.truncated_entropy(lam, k=9, norm=1)   # k clipped to d
    assert abs(H - 1.75 * math.log(2)) < 1e-14 and abs(E - 2 ** 1.75) < 1e-12
    # negative round-off eigenvalues count as zero
    H2, _ = oracle.truncated_entropy(np.array([1.0, -1e-18]), k=2)
    assert H2 == 0.0


def test_entropy_bounds_and_truncation_chain():
    # 0 <= H_k <= ln k ; 1 <= erank_k <= erank <= rank <= D (trace-normalised chain of the appendix)
    from paper_2410_03090_b200 import synth
    wl = synth.scaled(synth.WORKLOADS["c2"], N=384, L=1)
    for h in range(wl.H):
        K, _, _ = synth.generate_unit(wl, 0, 0, h)
        X = K.double().numpy()
        for k in (4, 32, 128):
            H, E = oracle.entropy(X, k_trunc=k, norm=0)
            assert -1e-12 <= H <= math.log(k) + 1e-12
            assert 1.0 - 1e-12 <= E <= k + 1e-9
        Hk, Ek = oracle.entropy(X, k_trunc=32, norm=1)
        Hf, Ef = oracle.entropy(X, k_trunc=128, norm=1)
        assert 1.0 - 1e-12 <= Ek <= Ef + 1e-12 <= 128 + 1e-9


def test_entropy_invariances():
    X = RNG.normal(size=(96, 16)) @ np.diag(np.linspace(0.1, 3.0, 16))
    H0, _ = oracle.entropy(X, k_trunc=6)
    assert abs(oracle.entropy(3.7 * X, k_trunc=6)[0] - H0) < 1e-12                   # scale
    assert abs(oracle.entropy(X[RNG.permutation(96)], k_trunc=6)[0] - H0) < 1e-12     # token order
    assert abs(oracle.entropy(X @ _orthogonal(16), k_trunc=6)[0] - H0) < 1e-11        # feature rotation
    assert abs(oracle.entropy(X + RNG.normal(size=(1, 16)), k_trunc=6)[0] - H0) < 1e-11  # constant row (centred)
    # and the uncentred variant is *not* invariant to a constant row
    Hu = oracle.entropy(X, k_trunc=6, center=False)[0]
    assert abs(oracle.entropy(X + 5.0, k_trunc=6, center=False)[0] - Hu) > 1e-3


def test_entropy_eigen_form_equals_trace_form():
    # Lemma 2: -sum sigma ln sigma equals -Tr(S ln S) for unit-trace S; matrix log via LAPACK eigenvectors
    X = RNG.normal(size=(50, 6))
    S = oracle.covariance(X)
    S /= np.trace(S)
    wv, V = np.linalg.eigh(S)
    logS = (V * np.log(wv)) @ V.T
    H, _ = oracle.truncated_entropy(oracle.eigenvalues(S), k=6, norm=1)
    assert abs(H + np.trace(S @ logS)) < 1e-12
