"""Shared checks for the GPU parity tests: CUDA path (through the C ABI) vs the fp64 oracle.

Bars: masks and packed indices bit-exact except for
draws within 1e-6 of their probability (counted and reported); singular values, probabilities
and decoded gradients within 1e-4 relative l2 / Frobenius error.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor

import numpy as np

REL_TOL = 1e-4          # relative l2 / Frobenius bar for floating-point results
CARVE = 1e-6            # |u_i - p_i| below this: the draw is excluded from bit-exactness
RESID_GRAM = 6e-7       # eigen-residual bar of the fp32 Gram route, in units of lambda_1 = sigma_1^2:
                        # twice the Jacobi rotation threshold (3e-7), i.e. about 10 ulp of fp32
GAP_MIN = 1e-3          # an atom's rank-one term is comparable across two SVDs only if
                        # min_j |sigma_i^2 - sigma_j^2| >= GAP_MIN * sigma_1^2 (well-conditioned).  The bound is the
                        # Gram matrix's, not the eigen-solver's: A = G G^T is stored in fp32, a perturbation E of
                        # about 1e-7 lambda_1, and an eigenvector moves by ||E|| / gap; 1e-7 / 1e-3 = 1e-4 is the
                        # bar for the decoded gradient.  Every test prints the largest (term error x gap) it saw.

# Calibrated per route and size (tests/test_gpu_gap_certificate.py measures err <= floor + c / gap on seeds of its own):
# on the tridiagonal routes the vectors come from an fp64 factorisation of T, and c is 2e-10 ... 4e-10 up to a short side
# of 512 (fp64 reduction) and 9e-9 at 1024 (fp32 storage): a gap of 4e-6 resp. 9e-5 would do for the 1e-4 bar; the values
# below keep a factor of 2.5 to 3 on top.  The Jacobi routes and short sides above 1024 keep the Gram matrix's own bound.
GAP_MIN_TRIDIAG_512 = 1e-5
GAP_MIN_TRIDIAG_1024 = 3e-4


def gap_min_for(short_side, eigen_scheme):
    """Smallest relative gap at which a kept atom's rank-one term is compared with the oracle's."""
    if eigen_scheme == 3 and short_side <= 512:
        return GAP_MIN_TRIDIAG_512
    if eigen_scheme == 3 and short_side <= 1024:
        return GAP_MIN_TRIDIAG_1024
    return GAP_MIN


# what the spectral checks of this session have compared so far (printed and asserted by the tests)
TALLY = {"layers": 0, "masks_identical": 0, "kept_atoms": 0, "certified_atoms": 0, "terms_compared": 0,
         "decodes_compared": 0, "worst_err_times_gap": 0.0}


def rel(a, b):
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    d = np.linalg.norm(a - b)
    n = np.linalg.norm(b)
    return d / n if n > 0 else d


def near_threshold(enc):
    u = enc["words"].astype(np.float64) / 2.0 ** 32
    return np.abs(u - enc["p"]) <= CARVE


def check_masks(mask_gpu, enc, report, tag):
    near = near_threshold(enc)
    diff = mask_gpu != enc["mask"]
    report.append(f"{tag}: draws within {CARVE:g} of p: {int(near.sum())}, differing masks among them: "
                  f"{int((diff & near).sum())}")
    assert not np.any(diff & ~near), f"{tag}: mask differs outside the carve-out at {np.flatnonzero(diff & ~near)[:8]}"
    return not diff.any()


def check_entrywise(A, oracle, g_np, g_dev, s, seed, step, layer_arrays, hdr, dbg, l, report, tag):
    """One vector of an entry-wise encode against the oracle.  Returns True if masks were identical."""
    n = g_np.size
    enc = oracle.encode_entrywise(g_np, s, seed, step=step, layer=l)
    assert hdr.status == 0, f"{tag}: status {hdr.status}"
    p = dbg.layer_prob(l, n)
    m = dbg.layer_mask(l, n)
    assert rel(p, enc["p"]) <= REL_TOL, f"{tag}: p rel {rel(p, enc['p'])}"
    assert np.abs(p - enc["p"]).max() <= 1e-6, f"{tag}: p max abs"
    same = check_masks(m, enc, report, tag)
    assert hdr.k == int(m.sum())
    assert np.array_equal(layer_arrays["idx"], np.flatnonzero(m).astype(np.uint32)), f"{tag}: packed indices"
    # saturated atoms: the same count, except that atoms sitting exactly on the boundary |lambda_i| (s - n_s) = tail
    # (p_i = 1 on either branch of Algorithm 1) may be counted on either side
    ties = int(np.count_nonzero(enc["p"] == 1.0)) - enc["n_s"]
    assert enc["n_s"] <= int(hdr.n_sat) <= enc["n_s"] + max(ties, 0), f"{tag}: n_sat {hdr.n_sat} vs {enc['n_s']} (+{ties} ties)"
    assert abs(hdr.l1 - np.abs(g_np.astype(np.float64)).sum()) <= 1e-7 * max(hdr.l1, 1e-300)
    # values: g_i / p_i with the oracle's p
    idx = layer_arrays["idx"].astype(np.int64)
    want = g_np.astype(np.float64)[idx] / enc["p"][idx]
    assert rel(layer_arrays["val"], want) <= REL_TOL, f"{tag}: values"
    return same, enc


def oracle_spectral_batch(oracle, mats, s, seed, step, threads=8):
    def one(args):
        l, G = args
        return oracle.encode_spectral(G, s, seed, step=step, layer=l)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(one, list(enumerate(mats))))


def check_spectral_layer(oracle, G, enc, hdr, arr, dbg, l, out_gpu, report, tag, check_vectors=True, gap_min=None):
    """One layer of a spectral encode + decode against the oracle (P1-P8 of the test plan)."""
    G64 = G.astype(np.float64)
    m_, n_ = G.shape
    r = min(m_, n_)
    s1 = max(enc["sigma"][0], 1e-300)
    assert hdr.status == 0, f"{tag}: status {hdr.status}"
    sig = dbg.layer_sigma(l, r); p = dbg.layer_prob(l, r); mask = dbg.layer_mask(l, r)
    # P1 singular values, P2 probabilities
    assert rel(sig, enc["sigma"]) <= REL_TOL, f"{tag}: sigma rel {rel(sig, enc['sigma'])}"
    assert rel(p, enc["p"]) <= REL_TOL, f"{tag}: p rel {rel(p, enc['p'])}"
    assert np.all(p >= 0) and np.all(p <= 1)
    n_nz = int(np.count_nonzero(enc["sigma"] > 1e-7 * s1))
    assert abs(p.sum() - enc["p"].sum()) <= 1e-4 * max(enc["p"].sum(), 1)
    # P3 masks and packed ranks
    same = check_masks(mask, enc, report, tag)
    assert hdr.k == int(mask.sum()) and np.array_equal(arr["idx"], np.flatnonzero(mask).astype(np.uint32))
    k = arr["k"]
    # P4 every kept atom is a singular triplet in the backward sense
    for j in range(k):
        u = arr["U"][:, j].astype(np.float64); v = arr["V"][:, j].astype(np.float64)
        sg = float(arr["coef"][j]) * float(p[arr["idx"][j]])
        assert abs(np.linalg.norm(u) - 1) <= 1e-5 and abs(np.linalg.norm(v) - 1) <= 1e-5, f"{tag}: atom {j} not unit"
        # the long-side vector is the back-projection of the short-side one, so one residual is
        # rounding only; the other is the eigen-residual of the fp32 Gram matrix, ||A x - lambda x||
        # <= RESID_GRAM * lambda_1, seen through 1/sigma_i
        small, big = 2e-5 * s1, max(2e-5 * s1, RESID_GRAM * s1 * s1 / max(sg, 1e-300))
        r_u = np.linalg.norm(G64.T @ u - sg * v); r_v = np.linalg.norm(G64 @ v - sg * u)
        lo, hi = (r_u, r_v) if m_ <= n_ else (r_v, r_u)
        assert lo <= small, f"{tag}: atom {j} back-projection residual {lo / s1:.2e}"
        assert hi <= big, f"{tag}: atom {j} eigen residual {hi / s1:.2e} (sigma_i/sigma_1 = {sg / s1:.2e})"
        assert abs(sg - enc["sigma"][arr["idx"][j]]) <= 2e-5 * s1
    # P5 decode kernel alone: GPU decode of the GPU payload vs the oracle's decode of the same payload
    own = oracle.decode_spectral(arr["coef"], arr["U"], arr["V"])
    if k:
        assert rel(out_gpu, own) <= 1e-5, f"{tag}: decode kernel {rel(out_gpu, own)}"
    else:
        assert not out_gpu.any()
    # P7 end to end vs the oracle's own encode + decode.  Per kept atom: its rank-one term against the oracle's
    # where the atom is well conditioned (certified); the whole decoded gradient where every kept atom is.
    e2e = None
    TALLY["layers"] += 1
    if same:
        TALLY["masks_identical"] += 1
        ref = oracle.decode_spectral(enc["coef"], enc["U_S"], enc["V_S"])
        ref_norm = max(np.linalg.norm(ref), 1e-300)
        e2e = rel(out_gpu, ref) if k else 0.0
        lam = enc["sigma"] ** 2
        all_ok = True
        for j, i in enumerate(arr["idx"]):
            others = np.delete(lam, i)
            gap = np.min(np.abs(others - lam[i])) / lam[0] if others.size else 1.0
            ok = gap >= (GAP_MIN if gap_min is None else gap_min)
            all_ok &= ok
            TALLY["kept_atoms"] += 1
            term = float(arr["coef"][j]) * np.outer(arr["U"][:, j].astype(np.float64), arr["V"][:, j].astype(np.float64))
            term_ref = float(enc["coef"][j]) * np.outer(enc["U_S"][:, j], enc["V_S"][:, j])
            err = np.linalg.norm(term - term_ref) / ref_norm
            TALLY["worst_err_times_gap"] = max(TALLY["worst_err_times_gap"], float(err * gap))
            if ok and check_vectors:
                TALLY["certified_atoms"] += 1
                TALLY["terms_compared"] += 1
                assert err <= REL_TOL, f"{tag}: kept atom {j} (rank {i}, gap {gap:.1e}): term error {err:.2e}"
        report.append(f"{tag}: k={k} end-to-end rel Frobenius {e2e:.2e} ({'certified' if all_ok else 'ill-conditioned atoms'})")
        if all_ok and check_vectors:
            TALLY["decodes_compared"] += 1
            assert e2e <= REL_TOL, f"{tag}: end-to-end {e2e}"
    return same, e2e


def check_full_basis(G, dbg, l, tag, orth_tol=1e-3, recon_tol=1e-4):
    """P8: the short-side vectors form an orthonormal basis that reproduces G by projection."""
    r = min(G.shape)
    Us = dbg.layer_short(l, r).astype(np.float64)          # rank-major: row a = vector a
    assert np.abs(Us @ Us.T - np.eye(r)).max() <= orth_tol, f"{tag}: orthogonality {np.abs(Us @ Us.T - np.eye(r)).max()}"
    G64 = G.astype(np.float64)
    proj = (Us.T @ (Us @ G64)) if G.shape[0] <= G.shape[1] else ((G64 @ Us.T) @ Us)
    assert rel(proj, G64) <= recon_tol, f"{tag}: projection reproduces G to {rel(proj, G64)}"
