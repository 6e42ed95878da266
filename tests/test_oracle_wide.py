"""Pins of the wide-matrix entropy oracle (paper Section 3.1 Eq. 1, Section 3.2): it must agree with the
Jacobi-based oracle where both run, and with spectra planted by construction."""
import math

import numpy as np
import pytest

import oracle


def _orthonormal(rng, rows, cols):
    q, _ = np.linalg.qr(rng.standard_normal((rows, cols)))
    return q


def test_agrees_with_the_jacobi_oracle():
    rng = np.random.default_rng(0)
    X = rng.standard_normal((300, 6)) @ rng.standard_normal((6, 192)) + 0.05 * rng.standard_normal((300, 192))
    for center in (True, False):
        for norm in (0, 1):
            Hw, Ew, lw = oracle.entropy_wide(X, 16, center, norm, return_spectrum=True)
            Hj, Ej, lj = oracle.entropy(X, 16, center, norm, return_spectrum=True)
            assert abs(Hw - Hj) < 1e-10 and abs(Ew - Ej) < 1e-9
            np.testing.assert_allclose(lw[:16], lj[:16], rtol=1e-10)


def test_planted_spectrum_and_closed_forms():
    rng = np.random.default_rng(1)
    N, D, r = 700, 512, 40
    sig = np.sqrt(np.linspace(50.0, 1.0, r))
    ones = np.ones(N) / math.sqrt(N)
    U = rng.standard_normal((N, r))
    U -= np.outer(ones, ones @ U)                      # columns orthogonal to the all-ones vector: centring is a no-op
    U = np.linalg.qr(U)[0]                             # an orthonormal basis of the same subspace
    V = _orthonormal(rng, D, r)
    X = (U * sig) @ V.T
    H, E, lam = oracle.entropy_wide(X, 32, True, 0, return_spectrum=True)
    np.testing.assert_allclose(lam[:r], sig ** 2, rtol=1e-9)
    p = sig[:32] ** 2 / (sig[:32] ** 2).sum()
    assert abs(H - float(-(p * np.log(p)).sum())) < 1e-10 and abs(E - math.exp(H)) < 1e-9
    # whole-trace normalisation keeps the top-k terms of the full entropy sum
    pf = sig ** 2 / (sig ** 2).sum()
    assert abs(oracle.entropy_wide(X, 32, True, 1)[0] - float(-(pf[:32] * np.log(pf[:32])).sum())) < 1e-10
    # equal planted values: H_k = ln k;  one direction: H = 0
    Xi = U[:, :32] @ V[:, :32].T
    assert abs(oracle.entropy_wide(Xi, 32)[0] - math.log(32)) < 1e-9
    X1 = np.outer(U[:, 0], V[:, 0]) * 3.0
    assert abs(oracle.entropy_wide(X1, 32)[0]) < 1e-9


def test_centring_removes_a_common_offset_and_transposition_matters():
    rng = np.random.default_rng(2)
    X = rng.standard_normal((90, 160)) * np.linspace(3.0, 0.1, 160)
    H0 = oracle.entropy_wide(X, 24)[0]
    assert abs(oracle.entropy_wide(X + 7.5, 24)[0] - H0) < 1e-9            # Eq. 1 subtracts the mean row
    assert abs(oracle.entropy_wide(X + 7.5, 24, center=False)[0] - H0) > 1e-3
    # rows are tokens: centring over columns instead gives another answer
    assert abs(oracle.entropy_wide(X.T.copy(), 24)[0] - H0) > 1e-6
    # N < D: at most N - 1 non-zero eigenvalues after centring
    lam = oracle.entropy_wide(X, 24, return_spectrum=True)[2]
    assert lam[88] > 1e-9 * lam[0] and abs(lam[89]) < 1e-9 * lam[0]
