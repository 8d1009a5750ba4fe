"""The stored oracle results for the large spectral layers, checked against what does not come from the
oracle's own SVD: the seeded input (CRC), a library SVD in fp64, the defining relations of a singular
triplet, and Algorithm 1 / Eq. 2 recomputed from the stored singular values."""
import numpy as np
import pytest

from tests import golden_io

CASES = [("c5small", 0), ("c5", 0), ("c5", 1), ("c3", 8)]


@pytest.mark.parametrize("case,index", CASES)
def test_stored_case(oracle, case, index):
    if not golden_io.have(case, index):
        pytest.skip("stored case not generated")
    G, meta, encs = golden_io.load(case, index)          # asserts shape and CRC of the regenerated input
    G64 = G.astype(np.float64)
    r = min(G.shape)
    sigma = next(iter(encs.values()))["sigma"]
    assert sigma.shape == (r,) and np.all(np.diff(sigma) <= 0) and sigma[-1] >= 0
    ref = np.linalg.svd(G64, compute_uv=False)
    assert np.abs(sigma - ref).max() <= 1e-12 * ref[0]
    assert abs(np.sum(sigma ** 2) - np.sum(G64 ** 2)) <= 1e-12 * np.sum(G64 ** 2)
    for s, enc in encs.items():
        p, n_s, _ = oracle.atomo_probabilities(sigma, s)
        assert np.array_equal(p, enc["p"]) and n_s == enc["n_s"]
        assert abs(p.sum() - min(s, r)) <= 1e-12 * s
        words = oracle.bernoulli_words(meta["philox_seed"], meta["step"], meta["layer"], oracle.KIND_SPECTRAL, r)
        mask = oracle.sample_mask(p, words)
        assert np.array_equal(mask, enc["mask"]) and np.array_equal(np.flatnonzero(mask), enc["idx"])
        assert np.allclose(enc["coef"], sigma[enc["idx"]] / p[enc["idx"]], rtol=0, atol=0)
        for j, i in enumerate(enc["idx"]):
            u, v = enc["U_S"][:, j], enc["V_S"][:, j]
            assert abs(np.linalg.norm(u) - 1) <= 1e-12 and abs(np.linalg.norm(v) - 1) <= 1e-12
            assert np.linalg.norm(G64 @ v - sigma[i] * u) <= 1e-11 * ref[0]
            assert np.linalg.norm(G64.T @ u - sigma[i] * v) <= 1e-11 * ref[0]
