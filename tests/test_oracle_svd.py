"""Pins for the oracle's one-sided Jacobi SVD (Section 5; Appendix C's tight examples)."""
import numpy as np
import pytest

from paper_1806_04090_b200 import synth


def _check_svd(X, U, sig, V, tol=1e-12):
    m, n = X.shape
    r = min(m, n)
    assert U.shape == (m, r) and V.shape == (n, r) and sig.shape == (r,)
    assert np.all(np.diff(sig) <= 0) and np.all(sig >= 0)
    scale = max(np.linalg.norm(X), 1e-300)
    assert np.linalg.norm((U * sig) @ V.T - X) <= tol * scale
    live = sig > 1e-13 * max(sig[0], 1e-300)
    Ul, Vl = U[:, live], V[:, live]
    assert np.abs(Ul.T @ Ul - np.eye(Ul.shape[1])).max() <= tol * 10
    assert np.abs(Vl.T @ Vl - np.eye(Vl.shape[1])).max() <= tol * 10


@pytest.mark.parametrize("shape", [(7, 7), (5, 19), (23, 4), (1, 6), (6, 1), (40, 64)])
def test_matches_definition_and_library(oracle, shape):
    rng = np.random.default_rng(sum(shape))
    X = rng.standard_normal(shape)
    U, sig, V = oracle.jacobi_svd(X)
    _check_svd(X, U, sig, V)
    # third opinion: a library SVD (never linked into the oracle or the product)
    np.testing.assert_allclose(sig, np.linalg.svd(X, compute_uv=False), rtol=1e-12, atol=1e-14)
    # sum sigma^2 = ||X||_F^2 ; Lemma 8: ||X||_{1,1}/sqrt(nm) <= ||X||_* <= ||X||_{1,1}
    assert abs(np.sum(sig ** 2) - np.sum(X * X)) <= 1e-12 * np.sum(X * X)
    l11 = np.abs(X).sum()
    assert l11 / np.sqrt(X.size) <= sig.sum() * (1 + 1e-12) and sig.sum() <= l11 * (1 + 1e-12)


def test_prescribed_spectrum_is_recovered(oracle):
    # a matrix built as U diag(sigma) V^T with Haar factors returns that sigma and those
    # rank-one terms (the factors are fixed up to a joint sign)
    rng = np.random.default_rng(3)
    m, n = 12, 30
    sigma = np.arange(1, m + 1, dtype=np.float64) ** -1.5
    U0 = synth.haar_columns(rng, m, m); V0 = synth.haar_columns(rng, n, m)
    X = (U0 * sigma) @ V0.T
    U, sig, V = oracle.jacobi_svd(X)
    np.testing.assert_allclose(sig, sigma, rtol=1e-12)
    for i in range(m):
        np.testing.assert_allclose(np.outer(U[:, i], V[:, i]), np.outer(U0[:, i], V0[:, i]), atol=1e-10)
    # and for the transposed (tall) problem
    U, sig, V = oracle.jacobi_svd(X.T)
    np.testing.assert_allclose(sig, sigma, rtol=1e-12)
    np.testing.assert_allclose(np.outer(U[:, 0], V[:, 0]), np.outer(V0[:, 0], U0[:, 0]), atol=1e-10)


def test_appendix_c_tight_examples(oracle):
    # one-hot matrix: a single singular value 1 (||X||_* = ||X||_{1,1} = 1)
    X = np.zeros((5, 8)); X[0, 0] = 1.0
    U, sig, V = oracle.jacobi_svd(X)
    assert sig[0] == pytest.approx(1.0, abs=1e-15) and np.all(sig[1:] == 0)
    np.testing.assert_allclose(np.outer(U[:, 0], V[:, 0]) * sig[0], X, atol=1e-15)
    # all-ones n x m: a single singular value sqrt(nm)
    X = np.ones((6, 11))
    U, sig, V = oracle.jacobi_svd(X)
    assert sig[0] == pytest.approx(np.sqrt(66.0), rel=1e-14)
    assert np.all(sig[1:] <= 1e-14 * sig[0])
    np.testing.assert_allclose((U[:, :1] * sig[0]) @ V[:, :1].T, X, atol=1e-13)


def test_zero_matrix(oracle):
    U, sig, V = oracle.jacobi_svd(np.zeros((4, 9)))
    assert np.all(sig == 0) and not V.any()


def test_sign_convention_and_order(oracle):
    rng = np.random.default_rng(8)
    X = rng.standard_normal((9, 14))
    U, sig, V = oracle.jacobi_svd(X)
    for i in range(9):
        assert U[np.argmax(np.abs(U[:, i])), i] > 0


def test_config_shaped_layer(oracle):
    G = synth.c2_resnet18(seed=0, layers=synth.RESNET18_LAYERS[:2])
    for X in G:
        X = X.astype(np.float64)
        U, sig, V = oracle.jacobi_svd(X)
        _check_svd(X, U, sig, V)
        np.testing.assert_allclose(sig, np.linalg.svd(X, compute_uv=False), rtol=1e-11, atol=1e-15)


def test_spectral_encode_atoms(oracle):
    # Eq. (2) with SVD atoms: kept ranks carry sigma_i / p_i and their own singular vectors
    G = synth.c1_spectral(seed=1).astype(np.float64)
    enc = oracle.encode_spectral(G, 2.0, seed=3)
    k = enc["idx"]
    np.testing.assert_allclose(enc["coef"] * enc["p"][k], enc["sigma"][k], rtol=1e-14)
    for j, i in enumerate(k):
        np.testing.assert_allclose(G @ enc["V_S"][:, j], enc["sigma"][i] * enc["U_S"][:, j], atol=1e-12)
    assert abs(enc["p"].sum() - 2.0) < 1e-12
