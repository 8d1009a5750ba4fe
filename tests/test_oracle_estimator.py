"""Pins for the oracle's sampling, encode and decode: Philox known answers, the integer
Bernoulli decision, Lemma 1's moments by Monte Carlo, Table 1's second moments."""
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_philox_known_answers(oracle):
    n = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        out = oracle.philox4x32_10([w[0]], [w[1]], [w[2]], [w[3]], w[4], w[5])
        assert [int(o[0]) for o in out] == w[6:10]
        n += 1
    assert n == 3


def test_counter_layout(oracle):
    # atom i uses word i&3 of block i>>2; layer, step and kind select disjoint streams
    seed = 0x1234567887654321
    w = oracle.bernoulli_words(seed, step=5, layer=3, kind=1, n_atoms=11)
    for i in (0, 1, 5, 10):
        blk = oracle.philox4x32_10([i >> 2], [0], [3], [(1 << 31) | 5], seed & 0xFFFFFFFF, seed >> 32)
        assert int(w[i]) == int(blk[i & 3][0])
    base = oracle.bernoulli_words(seed, 5, 3, 1, 64)
    for other in (oracle.bernoulli_words(seed, 6, 3, 1, 64), oracle.bernoulli_words(seed, 5, 4, 1, 64),
                  oracle.bernoulli_words(seed, 5, 3, 0, 64), oracle.bernoulli_words(seed + 1, 5, 3, 1, 64)):
        assert np.count_nonzero(other == base) == 0
    # a prefix of a longer stream is the shorter stream (counter based, no state)
    assert np.array_equal(oracle.bernoulli_words(seed, 5, 3, 1, 1000)[:64], base)


def test_words_are_uniform(oracle):
    w = oracle.bernoulli_words(42, 0, 0, 1, 1 << 20).astype(np.float64) / 2.0 ** 32
    assert abs(w.mean() - 0.5) < 4 / np.sqrt(12 * w.size)
    hist = np.histogram(w, bins=64, range=(0, 1))[0]
    chi2 = np.sum((hist - w.size / 64) ** 2 / (w.size / 64))
    assert chi2 < 130          # 63 dof: mean 63, sd 11.2
    # lag-1 correlation
    assert abs(np.corrcoef(w[:-1], w[1:])[0, 1]) < 5 / np.sqrt(w.size)


def test_integer_decision(oracle):
    p = np.array([0.0, 1.0, 0.5, 0.5, 2.0 ** -32, 2.0 ** -32, 1 - 2.0 ** -33])
    x = np.array([0, 0xFFFFFFFF, 0x7FFFFFFF, 0x80000000, 0, 1, 0xFFFFFFFF], dtype=np.uint32)
    assert oracle.sample_mask(p, x).tolist() == [False, True, True, False, True, False, False]


@pytest.mark.parametrize("s", [1.5, 3.0])
def test_entrywise_moments_monte_carlo(oracle, s):
    # Lemma 1: E[g_hat] = g and E||g_hat||^2 = sum lambda_i^2 / p_i (orthonormal atoms)
    g = np.array([3.0, -1.0, 0.5, 0.0, 2.0, -0.25, 0.1])
    trials = 6000
    acc = np.zeros_like(g); acc2 = np.zeros_like(g); sq = 0.0; kept = 0
    for t in range(trials):
        enc = oracle.encode_entrywise(g, s, seed=1000 + t)
        gh = oracle.decode_entrywise(g.size, enc["idx"], enc["val"])
        acc += gh; acc2 += gh * gh; sq += gh @ gh; kept += enc["idx"].size
    p = enc["p"]
    mean = acc / trials
    var = np.where(p > 0, g ** 2 * (1 - p) / np.where(p > 0, p, 1), 0)
    assert np.all(np.abs(mean - g) <= 4.5 * np.sqrt(var / trials) + 1e-12)
    second = np.sum(g[p > 0] ** 2 / p[p > 0])
    assert abs(sq / trials - second) <= 0.05 * second
    # sparsity on average: E[#kept] = sum p = s
    assert abs(kept / trials - s) <= 4.5 * np.sqrt(np.sum(p * (1 - p)) / trials) + 1e-12


def test_spectral_moments_monte_carlo(oracle):
    # Lemma 1 with SVD atoms; Table 1: optimal second moment ||X||_*^2 / s when balanced.
    rng = np.random.default_rng(5)
    X = rng.standard_normal((6, 9))
    U, sig, V = oracle.jacobi_svd(X)
    s = 2.0
    assert s <= sig.sum() / sig.max()            # balanced (Lemma 3)
    trials = 4000
    acc = np.zeros_like(X); sq = 0.0; reals = 0
    for t in range(trials):
        enc = oracle.encode_spectral_from_svd(U, sig, V, s, seed=77 + t)
        Xh = oracle.decode_spectral(enc["coef"], enc["U_S"], enc["V_S"])
        acc += Xh; sq += np.sum(Xh * Xh); reals += enc["idx"].size * (X.shape[0] + X.shape[1])
    p = enc["p"]
    np.testing.assert_allclose(p, s * sig / sig.sum(), rtol=1e-12)
    # entry-wise standard error of the mean: Var(X_hat_ab) = sum_i sigma_i^2 (1-p_i)/p_i (u_ia v_ib)^2
    var = np.einsum("i,ai,bi->ab", sig ** 2 * (1 - p) / p, U ** 2, V ** 2)
    assert np.all(np.abs(acc / trials - X) <= 4.5 * np.sqrt(var / trials) + 1e-12)
    nuc2_over_s = sig.sum() ** 2 / s
    assert abs(sq / trials - nuc2_over_s) <= 0.05 * nuc2_over_s
    # Table 1: communication cost s (n + m) reals on average
    assert abs(reals / trials - s * (6 + 9)) <= 0.05 * s * 15


def test_table1_entrywise_second_moment(oracle):
    # Table 1: entry-wise optimum ||X||_{1,1}^2 / s when X is s-balanced entry-wise
    rng = np.random.default_rng(9)
    X = rng.standard_normal((5, 7))
    s = 4.0
    assert s <= np.abs(X).sum() / np.abs(X).max()
    p, _, _ = oracle.atomo_probabilities(X.reshape(-1), s)
    f = np.sum(X.reshape(-1) ** 2 / p)
    assert abs(f - np.abs(X).sum() ** 2 / s) <= 1e-10 * f


def test_decode_places_values(oracle):
    out = oracle.decode_entrywise(6, np.array([1, 4]), np.array([2.5, -3.0]))
    assert out.tolist() == [0, 2.5, 0, 0, -3.0, 0]
    assert oracle.decode_entrywise(3, np.array([], dtype=np.int64), np.array([])).tolist() == [0, 0, 0]
    z = oracle.decode_spectral(np.zeros(0), np.zeros((4, 0)), np.zeros((5, 0)))
    assert z.shape == (4, 5) and not z.any()
    # one atom: coef * u v^T, with the operands in the right places (u indexes rows)
    u = np.array([[1.0], [2.0]]); v = np.array([[1.0], [0.0], [-1.0]])
    np.testing.assert_array_equal(oracle.decode_spectral(np.array([2.0]), u, v),
                                  np.array([[2.0, 0, -2.0], [4.0, 0, -4.0]]))


def test_saturated_atoms_always_kept(oracle):
    g = np.array([100.0, 1.0, 1.0, 1.0, 1.0])
    for seed in range(50):
        enc = oracle.encode_entrywise(g, 2.0, seed)
        assert enc["mask"][0] and enc["val"][0] == 100.0      # p = 1: weight lambda / 1
