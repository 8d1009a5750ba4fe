"""The gap certificate of the end-to-end comparison, measured per size bucket on seeds of its own.

A kept atom's rank-one term can be compared between two SVDs only where the atom is well conditioned: the Gram matrix
is stored in fp32 (a perturbation of about 1e-7 lambda_1), and an eigenvector moves by that perturbation divided by the
gap of its eigenvalue to the nearest other one.  The parity checks therefore compare the terms of atoms whose gap is at
least a minimum (in units of lambda_1; parity.gap_min_for) to the 1e-4 bar.  This test measures the constant behind that rule: on the
default route, for short sides of 64 to 1024, with a budget large enough to keep atoms from the whole spectrum, it
records the term error and the gap of every kept atom against the oracle's term and fits err <= floor + c / gap: the
floor is the worst error among atoms with a gap of 0.1 or more (rounding of fp32 vectors, nothing to do with
conditioning), c the worst (err - floor) x gap among the others.  Per bucket it prints the number of atoms, how many
the gap in use certifies, floor, c, the gap that the 1e-4 bar really needs (c / (1e-4 - floor)) and the worst error among the
certified atoms.  Frozen bounds, with the gap of parity.gap_min_for (1e-5 up to a short side of 512, 3e-4 at 1024):
c <= gap x 1e-4 / 2 (the gap is sufficient with a factor of two to spare), floor <= 1e-5, and every atom the gap
certifies within 1e-4."""
import numpy as np
import pytest

from paper_1806_04090_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu

BUCKETS = [(64, 576, 16.0), (128, 1152, 24.0), (256, 2304, 32.0), (512, 4608, 32.0), (1024, 2048, 24.0)]
SEEDS = [101, 102, 103]


@pytest.fixture(scope="module")
def atomo():
    import torch
    from paper_1806_04090_b200 import api
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    a = api.Atomo(0)
    yield a
    a.close()


def test_gap_certificate_per_bucket(atomo, oracle):
    import torch
    rows = []
    for r, L, s in BUCKETS:
        pairs = []
        for seed in SEEDS[: (3 if r <= 512 else 1)]:                       # the oracle takes 20 s on a 1024 x 2048 matrix
            G = synth.lowrank_plus_noise(np.random.default_rng([r, seed]), r, L, 1.5, noise_rel=0.01)
            pay, _ = atomo.atomo_encode_spectral([torch.from_numpy(G).cuda()], s, seed, step=2, k_cap=min(r, 128), debug=True)
            hdrs = pay.headers()
            assert hdrs[1][0].status == 0
            arr = pay.layer_arrays(0, hdrs)
            enc = oracle.encode_spectral(G, s, seed, step=2, layer=0)
            if not np.array_equal(arr["idx"].astype(np.int64), np.flatnonzero(enc["mask"])):
                continue                                                    # a draw inside the carve-out: other atoms, nothing to pair up
            ref = oracle.decode_spectral(enc["coef"], enc["U_S"], enc["V_S"])
            ref_norm = max(np.linalg.norm(ref), 1e-300)
            lam = enc["sigma"] ** 2
            for j, i in enumerate(arr["idx"]):
                gap = np.min(np.abs(np.delete(lam, i) - lam[i])) / lam[0]
                term = float(arr["coef"][j]) * np.outer(arr["U"][:, j].astype(np.float64), arr["V"][:, j].astype(np.float64))
                term_ref = float(enc["coef"][j]) * np.outer(enc["U_S"][:, j], enc["V_S"][:, j])
                pairs.append((float(gap), float(np.linalg.norm(term - term_ref) / ref_norm)))
        assert pairs, f"short side {r}: no kept atoms were paired with the oracle's"
        wide = [e for g, e in pairs if g >= 0.1]
        floor = max(wide) if wide else 0.0
        c = max([max(e - floor, 0.0) * g for g, e in pairs if g < 0.1], default=0.0)
        cert = [e for g, e in pairs if g >= parity.gap_min_for(r, 3)]
        rows.append((r, L, s, len(pairs), len(cert), floor, c, c / (parity.REL_TOL - floor), max(cert, default=0.0)))
    print("\nshort side  long side  budget  kept atoms  certified by the gap     floor         c    gap needed for 1e-4  worst certified err")
    for row in rows:
        print("%10d %10d %7g %11d %21d %9.2e %9.2e %22.2e %20.2e" % row)
    for r, L, s, n_atoms, n_cert, floor, c, need, worst_cert in rows:
        assert floor <= 1e-5, f"short side {r}: error floor {floor:.2e}"
        assert c <= 0.5 * parity.gap_min_for(r, 3) * parity.REL_TOL, f"short side {r}: c = {c:.2e}: the gap in use is not sufficient"
        assert worst_cert <= parity.REL_TOL
