"""Pins for the oracle's Algorithm 1 against what the paper and the mathematics fix."""
import itertools
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _f(lam, p):
    lam = np.asarray(lam, dtype=np.float64)
    nz = lam != 0
    return float(np.sum(lam[nz] ** 2 / p[nz]))


def test_hand_cases(oracle):
    n_cases = 0
    for line in open(os.path.join(GOLDEN, "alg1_hand_cases.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        lam_s, s_s, p_s = [x.strip() for x in line.split(";")]
        lam = np.array([float(x) for x in lam_s.split(",")])
        p_exp = np.array([float(x) for x in p_s.split(",")])
        p, _, _ = oracle.atomo_probabilities(lam, float(s_s))
        np.testing.assert_allclose(p, p_exp, rtol=0, atol=1e-15, err_msg=line)
        n_cases += 1
    assert n_cases >= 10


@pytest.mark.parametrize("seed", range(20))
def test_budget_and_bounds(oracle, seed):
    # Eq. (3): sum p = s, 0 <= p <= 1; Appendix B: zero atoms get 0, p monotone in |lambda|,
    # at most ceil(s)-1 atoms are set to one before the test of Algorithm 1 holds.
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 400))
    lam = rng.standard_normal(n) * np.exp(3 * rng.standard_normal(n))
    lam[rng.random(n) < 0.2] = 0.0
    n_nz = int(np.count_nonzero(lam))
    s = float(rng.uniform(0.05, 1.3 * n))
    p, n_s, c = oracle.atomo_probabilities(lam, s)
    assert np.all(p >= 0) and np.all(p <= 1.0)
    assert np.all(p[lam == 0] == 0)
    assert abs(p.sum() - min(s, n_nz)) <= 1e-9 * max(s, 1)
    order = np.argsort(-np.abs(lam), kind="stable")
    assert np.all(np.diff(p[order]) <= 1e-15)
    if s < n_nz:
        assert n_s <= int(np.ceil(s)) - 1
        # unsaturated kept atoms all carry weight |lambda_i| / p_i = c
        unsat = (p < 1) & (lam != 0)
        np.testing.assert_allclose(np.abs(lam[unsat]) / p[unsat], c, rtol=1e-12)
        # lower bound of Appendix B: p_i >= s lambda_i^2 / (n ||lambda||_2^2)
        assert np.all(p >= s * lam ** 2 / (n * np.sum(lam ** 2)) - 1e-15)


@pytest.mark.parametrize("seed", range(10))
def test_balanced_closed_form(oracle, seed):
    # Lemma 2 / Lemma 3: s <= ||lambda||_1 / ||lambda||_inf  <=>  p_i = s |lambda_i| / ||lambda||_1
    rng = np.random.default_rng(100 + seed)
    lam = rng.standard_normal(int(rng.integers(2, 300)))
    a = np.abs(lam)
    s_max = a.sum() / a.max()
    for s in (0.3 * s_max, s_max * (1 - 1e-12)):
        p, n_s, c = oracle.atomo_probabilities(lam, s)
        np.testing.assert_allclose(p, s * a / a.sum(), rtol=1e-13)
        assert n_s == 0
        # Lemma 2: the optimum value is ||lambda||_1^2 / s
        assert abs(_f(lam, p) - a.sum() ** 2 / s) <= 1e-10 * a.sum() ** 2 / s
    # just beyond the balance limit the largest atom is unbalanced (Definition 1) -> p = 1
    p, n_s, _ = oracle.atomo_probabilities(lam, min(s_max * 1.01, lam.size))
    assert n_s >= 1 and p[np.argmax(a)] == 1.0


@pytest.mark.parametrize("seed", range(10))
def test_appendix_b_closed_form_first_feasible(oracle, seed):
    # Appendix B: n_s* is the FIRST n_s for which p_i = |l_i|(s-n_s)/sum_{j>n_s}|l_j| <= 1 for all i.
    rng = np.random.default_rng(200 + seed)
    n = int(rng.integers(3, 60))
    a = np.sort(np.abs(rng.standard_normal(n)) * np.exp(2 * rng.standard_normal(n)))[::-1]
    s = float(rng.uniform(1.0, n - 0.5))
    expect = None
    for n_s in range(n):
        rest = a[n_s:]
        cand = rest * (s - n_s) / rest.sum()
        if np.all(cand <= 1.0):
            expect = np.concatenate([np.ones(n_s), cand])
            break
    p, n_s_alg, _ = oracle.atomo_probabilities(a, s)
    np.testing.assert_allclose(p, expect, rtol=1e-12, atol=1e-15)


@pytest.mark.parametrize("seed", range(12))
def test_brute_force_optimum_small(oracle, seed):
    # Eq. (3) on <= 6 atoms: by the KKT conditions of Appendix B every optimum has p_i = 1 on
    # some subset S and p_i proportional to |lambda_i| elsewhere.  Enumerate ALL subsets (not
    # only "largest first"), keep the feasible candidates, and take the best.
    rng = np.random.default_rng(300 + seed)
    n = int(rng.integers(2, 7))
    lam = rng.standard_normal(n) * np.exp(1.5 * rng.standard_normal(n))
    a = np.abs(lam)
    s = float(rng.uniform(0.3, n - 0.05))
    best = np.inf
    for k in range(n):
        if s - k <= 0:
            break
        for S in itertools.combinations(range(n), k):
            rest = [i for i in range(n) if i not in S]
            p = np.ones(n)
            p[rest] = a[rest] * (s - k) / a[rest].sum()
            if np.all(p <= 1 + 1e-15):
                best = min(best, _f(lam, p))
    p_alg, _, _ = oracle.atomo_probabilities(lam, s)
    assert abs(_f(lam, p_alg) - best) <= 1e-10 * best
    # random feasible points never do better
    for _ in range(300):
        d = rng.standard_normal(n)
        d -= d.mean()
        q = p_alg + 0.05 * rng.random() * d
        if np.all(q > 0) and np.all(q <= 1):
            assert _f(lam, q) >= _f(lam, p_alg) * (1 - 1e-12)


@pytest.mark.parametrize("seed", range(4))
def test_against_constrained_minimiser(oracle, seed):
    # third opinion: a general-purpose constrained minimiser on Eq. (3)
    from scipy.optimize import minimize
    rng = np.random.default_rng(400 + seed)
    n = 5
    lam = rng.standard_normal(n) * np.array([6.0, 3.0, 1.0, 1.0, 0.5])
    s = 2.5
    res = minimize(lambda p: np.sum(lam ** 2 / p), np.full(n, s / n), method="SLSQP",
                   bounds=[(1e-9, 1.0)] * n,
                   constraints=[{"type": "eq", "fun": lambda p: p.sum() - s}],
                   options={"ftol": 1e-14, "maxiter": 500})
    p_alg, _, _ = oracle.atomo_probabilities(lam, s)
    assert _f(lam, p_alg) <= res.fun * (1 + 1e-9)
    np.testing.assert_allclose(p_alg, res.x, atol=2e-4)


def test_qsgd_terngrad_lq_special_cases(oracle):
    # Section 4: with s = ||g||_1 / ||g||_q the optimum is p_i = |g_i| / ||g||_q, the kept
    # entries decode to ||g||_q sign(g_i), and E||L_q(g)||^2 = ||g||_1 ||g||_q  (Theorem 6).
    rng = np.random.default_rng(7)
    g = rng.standard_normal(257)
    l1 = np.abs(g).sum()
    for q, nq in ((2, np.linalg.norm(g)), (np.inf, np.abs(g).max()), (3, np.sum(np.abs(g) ** 3) ** (1 / 3))):
        s = l1 / nq
        p, n_s, c = oracle.atomo_probabilities(g, s)
        np.testing.assert_allclose(p, np.abs(g) / nq, rtol=1e-12)
        assert abs(_f(g, p) - l1 * nq) <= 1e-10 * l1 * nq
        enc = oracle.encode_entrywise(g, s, seed=11)
        np.testing.assert_allclose(enc["val"], nq * np.sign(g[enc["idx"]]), rtol=1e-12)
        if q == np.inf:
            assert p[np.argmax(np.abs(g))] == pytest.approx(1.0, abs=1e-15)
            assert enc["mask"][np.argmax(np.abs(g))] or p[np.argmax(np.abs(g))] < 1.0


def test_lq_budget_pins(oracle):
    # closed forms: a one-hot vector has every norm equal; n equal entries give n^(1 - 1/q)
    hot = np.zeros(9); hot[4] = -3.5
    for q in (1.0, 1.5, 2.0, 7.0, np.inf):
        assert oracle.lq_budget(hot, q) == pytest.approx(1.0, rel=1e-15)
        flat = np.full(64, -0.25)
        want = 64.0 if np.isinf(q) else 64.0 ** (1.0 - 1.0 / q)
        assert oracle.lq_budget(flat, q) == pytest.approx(want, rel=1e-13)
    assert oracle.lq_budget(np.zeros(5), 2.0) == 0.0
    g = np.array([3.0, -4.0, 0.0, 12.0])
    assert oracle.lq_budget(g, 1.0) == pytest.approx(1.0, rel=1e-15)
    assert oracle.lq_budget(g, 2.0) == pytest.approx(19.0 / 13.0, rel=1e-15)       # ||g||_2 = 13
    assert oracle.lq_budget(g, np.inf) == pytest.approx(19.0 / 12.0, rel=1e-15)
    with pytest.raises(ValueError):
        oracle.lq_budget(g, 0.5)
    # Section 4: at this budget every vector is s-balanced and Algorithm 1 returns p_i = |g_i| / ||g||_q
    rng = np.random.default_rng(12)
    for q in (2.0, 3.0, np.inf):
        g = rng.standard_normal(500) * np.exp(rng.standard_normal(500))
        s = oracle.lq_budget(g, q)
        nq = np.abs(g).max() if np.isinf(q) else (np.abs(g) ** q).sum() ** (1.0 / q)
        p, n_s, _ = oracle.atomo_probabilities(g, s)
        assert n_s == 0
        np.testing.assert_allclose(p, np.abs(g) / nq, rtol=1e-12, atol=0)


def test_budget_errors(oracle):
    for bad in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(ValueError):
            oracle.atomo_probabilities([1.0, 2.0], bad)


def test_all_zero_and_empty(oracle):
    p, n_s, c = oracle.atomo_probabilities(np.zeros(5), 2.0)
    assert np.all(p == 0) and c == 0.0
    p, n_s, c = oracle.atomo_probabilities(np.zeros(0), 2.0)
    assert p.size == 0
