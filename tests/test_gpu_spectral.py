"""GPU parity: spectral ATOMO through the C ABI vs the fp64 oracle."""
import numpy as np
import pytest

from paper_1806_04090_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def atomo():
    import torch
    from paper_1806_04090_b200 import api
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    a = api.Atomo(0)
    yield a
    a.close()


def _encode(atomo, mats, s, seed, step=0, k_cap=None, pad_ld=0):
    import torch
    ts = []
    for G in mats:
        if pad_ld:
            buf = torch.full((G.shape[0], G.shape[1] + pad_ld), 7.0, dtype=torch.float32, device="cuda")
            buf[:, : G.shape[1]] = torch.from_numpy(G).cuda()
            ts.append(buf[:, : G.shape[1]])
        else:
            ts.append(torch.from_numpy(G).cuda())
    if k_cap is None:
        k_cap = max(min(G.shape) for G in mats)
    pay, dbg = atomo.atomo_encode_spectral(ts, s, seed, step=step, k_cap=k_cap, debug=True, debug_short=True)
    return pay, dbg


def _run(atomo, oracle, mats, s, seed, step=0, pad_ld=0, check_vectors=True, orth_tol=1e-3):
    pay, dbg = _encode(atomo, mats, s, seed, step, pad_ld=pad_ld)
    hdrs = pay.headers()
    outs = atomo.atomo_decode(pay)
    encs = parity.oracle_spectral_batch(oracle, mats, s, seed, step)
    report = []
    n_same = 0
    for l, G in enumerate(mats):
        arr = pay.layer_arrays(l, hdrs)
        out = outs[l].cpu().numpy().astype(np.float64)
        same, _ = parity.check_spectral_layer(oracle, G, encs[l], hdrs[1][l], arr, dbg, l, out, report,
                                              f"L{l}{G.shape}", check_vectors)
        parity.check_full_basis(G, dbg, l, f"L{l}{G.shape}", orth_tol=orth_tol)
        n_same += same
    print("\n".join(report))
    print(f"layers with identical masks: {n_same}/{len(mats)}; sweeps: {[h.sweeps for h in hdrs[1]]}")
    return pay, hdrs, encs


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_config1_spectral(atomo, oracle, seed):
    _run(atomo, oracle, [synth.c1_spectral(seed)], 2.0, seed=11 + seed, step=1)


@pytest.mark.parametrize("shape", [(1, 1), (1, 9), (7, 1), (3, 5), (5, 3), (10, 512), (64, 27), (33, 100), (100, 33),
                                   (65, 130), (130, 257)])
def test_small_and_ragged_shapes(atomo, oracle, shape):
    rng = np.random.default_rng(sum(shape))
    G = synth.lowrank_plus_noise(rng, shape[0], shape[1], 1.0, noise_rel=0.05)
    _run(atomo, oracle, [G], 1.5, seed=21)


def test_saturating_budget(atomo, oracle):
    # fc 10 x 512 of the ResNet-18 set: sum(sigma) < 2 sigma_1, the top atom gets p = 1
    G = synth.c2_resnet18(0, [synth.RESNET18_LAYERS[17]])[0]
    pay, hdrs, encs = _run(atomo, oracle, [G], 2.0, seed=5)
    assert hdrs[1][0].n_sat == 1 == encs[0]["n_s"]
    # s >= number of atoms: everything kept, decode reproduces G (no sparsification)
    pay, hdrs, _ = _run(atomo, oracle, [G], 10.0, seed=5)
    assert hdrs[1][0].k == 10
    out = atomo.atomo_decode(pay)[0].cpu().numpy()
    assert parity.rel(out, G) <= 1e-5


def test_rank_deficient_inputs(atomo, oracle):
    import torch
    ones = np.ones((6, 11), dtype=np.float32)          # single singular value sqrt(66)
    hot = np.zeros((5, 8), dtype=np.float32); hot[0, 0] = 1.0
    zero = np.zeros((4, 9), dtype=np.float32)
    pay, dbg = _encode(atomo, [ones, hot, zero], 1.0, seed=3)
    hdrs = pay.headers()
    assert [h.status for h in hdrs[1]] == [0, 0, 0]
    sig = dbg.layer_sigma(0, 6)
    assert abs(sig[0] - np.sqrt(66.0)) <= 1e-5 * np.sqrt(66.0) and np.all(sig[1:] <= 1e-3)
    sig = dbg.layer_sigma(1, 5)
    assert abs(sig[0] - 1.0) <= 1e-6 and np.all(sig[1:] <= 1e-6)
    outs = atomo.atomo_decode(pay)
    assert hdrs[1][2].k == 0 and not outs[2].any()
    # budget 1 on a rank-one matrix: the atom has p = 1 and decode returns the matrix
    assert parity.rel(outs[0].cpu().numpy(), ones) <= 1e-5
    assert parity.rel(outs[1].cpu().numpy(), hot) <= 1e-5


def test_batch_mixed_sizes(atomo, oracle):
    L = synth.RESNET18_LAYERS
    mats = synth.c2_resnet18(0, [L[0], L[1], L[5], L[6], L[9], L[17]])
    _run(atomo, oracle, mats, 2.0, seed=3, step=4)


def test_paper_reshape_family(atomo, oracle):
    # Section 6 matricises a conv gradient (x, y, k, k) as x*y/2 rows by 2 k^2 = 18 columns: very tall layers
    mats = synth.c2_paper_reshape(0)
    assert [m.shape for m in mats] == [(96, 18), (2048, 18), (4096, 18), (16384, 18)]
    _run(atomo, oracle, mats, 2.0, seed=17, step=1)


@pytest.mark.parametrize("scheme", [0, 1, 2])
def test_jacobi_launch_schemes_against_oracle(atomo, oracle, scheme):
    """Each launch form of the Jacobi fallback (one launch per step, persistent cooperative launches, clusters)
    directly against the oracle, full protocol."""
    L = synth.RESNET18_LAYERS
    mats = synth.c2_resnet18(3, [L[0], L[1], L[5], L[9], L[17]])
    try:
        atomo.set_persistent_eig(scheme)
        _run(atomo, oracle, mats, 2.0, seed=77, step=3)
        assert atomo.last_eig_scheme() == scheme
    finally:
        atomo.set_persistent_eig(3)


def test_eigen_launch_schemes_agree(atomo):
    """One launch per step, persistent cooperative launches and the cluster form run the same rotations in the same
    order per layer: identical masks and singular values to rounding (the forms fold the row factors at different
    moments, so the bits may differ)."""
    L = synth.RESNET18_LAYERS
    mats = synth.c2_resnet18(1, [L[0], L[1], L[5], L[9], L[13], L[17]])
    got = []
    try:
        for scheme in (0, 1, 2):
            atomo.set_persistent_eig(scheme)
            pay, dbg = _encode(atomo, mats, 2.0, seed=23, step=2)
            hdrs = pay.headers()[1]
            assert [h.status for h in hdrs] == [0] * len(mats)
            got.append(([dbg.layer_sigma(l, min(m.shape)) for l, m in enumerate(mats)],
                        [pay.layer_arrays(l)["idx"].copy() for l in range(len(mats))]))
    finally:
        atomo.set_persistent_eig(3)
    for other in got[1:]:
        for l in range(len(mats)):
            assert parity.rel(other[0][l], got[0][0][l]) <= 2e-6
            assert np.array_equal(other[1][l], got[0][1][l])


def test_random_batches(atomo):
    """Seeded random batches (1 to 39 layers, short sides 1 to 512, wide and tall, several spectra, noise levels and
    budgets): the packing of layers into clusters, idle CTAs, tiny and ragged layers.  Properties that hold at any
    size: status, singular values against a library SVD, sum(p) = min(s, rank), decode = its definition."""
    import torch
    rng = np.random.default_rng(77)
    for trial in range(8):
        n_layers = int(rng.integers(1, 40))
        mats = []
        for l in range(n_layers):
            m = int(rng.choice([1, 3, 10, 17, 33, 64, 100, 129, 200, 256, 300, 512]))
            n = int(rng.choice([1, 5, 18, 27, 64, 130, 576, 700, 1152]))
            if rng.random() < 0.3:
                m, n = n, m
            mats.append(synth.lowrank_plus_noise(np.random.default_rng([trial, l]), m, n, float(rng.choice([0.5, 1.0, 1.5])),
                                                 noise_rel=float(rng.choice([0.0, 0.01, 0.1]))))
        s = float(rng.choice([0.5, 1.0, 2.0, 3.7]))
        ts = [torch.from_numpy(G).cuda() for G in mats]
        pay, dbg = atomo.atomo_encode_spectral(ts, s, seed=trial, step=trial, k_cap=64, debug=True)
        hdrs = pay.headers()
        assert [h.status for h in hdrs[1]] == [0] * n_layers
        outs = atomo.atomo_decode(pay)
        for l, G in enumerate(mats):
            r = min(G.shape)
            ref = np.linalg.svd(G.astype(np.float64), compute_uv=False)
            sig = dbg.layer_sigma(l, r)
            assert parity.rel(sig, ref) <= parity.REL_TOL, (trial, l, G.shape)
            p = dbg.layer_prob(l, r)
            assert abs(p.sum() - min(s, float((sig > 0).sum()))) <= 1e-3 * max(s, 1.0), (trial, l, G.shape)
            arr = pay.layer_arrays(l, hdrs)
            out = outs[l].cpu().numpy()
            if arr["k"]:
                own = (arr["U"].astype(np.float64) * arr["coef"].astype(np.float64)) @ arr["V"].astype(np.float64).T
                assert parity.rel(out, own) <= 1e-5, (trial, l, G.shape)
            else:
                assert not out.any()


def test_leading_dimension(atomo, oracle):
    rng = np.random.default_rng(7)
    mats = [synth.lowrank_plus_noise(rng, 48, 200, 1.0, noise_rel=0.02),
            synth.lowrank_plus_noise(rng, 150, 40, 1.0, noise_rel=0.02)]
    _run(atomo, oracle, mats, 2.0, seed=13, pad_ld=5)


def test_deterministic(atomo):
    G = synth.c2_resnet18(1, [synth.RESNET18_LAYERS[6]])
    p1, _ = _encode(atomo, G, 2.0, seed=9)
    p2, _ = _encode(atomo, G, 2.0, seed=9)
    a1, a2 = p1.layer_arrays(0), p2.layer_arrays(0)
    for key in ("idx", "coef", "U", "V"):
        assert np.array_equal(a1[key], a2[key])


def test_device_side_errors(atomo):
    import torch
    G = synth.c1_spectral(0).copy()
    t = torch.from_numpy(G).cuda()
    pay, _ = atomo.atomo_encode_spectral([t], 40.0, seed=1, k_cap=4)       # about 40 atoms kept > 4
    assert atomo.payload_status(pay) == (3, 0)
    assert pay.headers()[1][0].k == 0 and not atomo.atomo_decode(pay)[0].any()
    G[3, 3] = np.nan
    pay, _ = atomo.atomo_encode_spectral([torch.from_numpy(G).cuda()], 2.0, seed=1, k_cap=64)
    assert atomo.payload_status(pay) == (4, 0) and pay.headers()[1][0].k == 0
    assert not atomo.atomo_decode(pay)[0].any()


def test_host_side_errors(atomo):
    import torch
    from paper_1806_04090_b200 import api
    t = torch.ones(8, 8, device="cuda")
    for bad in (0.0, -1.0, float("nan")):
        with pytest.raises(api.AtomoError) as e:
            atomo.atomo_encode_spectral([t], bad, seed=1)
        assert e.value.code == 2
    with pytest.raises(api.AtomoError) as e:
        atomo.atomo_encode_spectral([t], 2.0, seed=1, k_cap=8, payload=torch.empty(128, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 3


def test_sweep_cap_reports_not_converged(atomo):
    # a bounded eigen-solver: with the cap at one sweep the layer reports NOT_CONVERGED (no trap, no hang).
    # Route 1 (rows orthogonal only at convergence) then keeps nothing; route 0 keeps its orthonormal basis.
    import torch
    G = synth.c2_resnet18(0, [synth.RESNET18_LAYERS[5]])[0]
    t = torch.from_numpy(G).cuda()
    atomo.set_eig_params(1, 3e-7)
    atomo.set_persistent_eig(2)                       # the Jacobi routes are the iterative ones (the tridiagonal route has no sweeps)
    try:
        pay, _ = atomo.atomo_encode_spectral([t], 2.0, seed=1, k_cap=128)
        assert atomo.payload_status(pay) == (5, 0) and pay.headers()[1][0].k == 0
        assert not atomo.atomo_decode(pay)[0].any()
        atomo.set_eig_mode(0)
        pay, dbg = atomo.atomo_encode_spectral([t], 2.0, seed=1, k_cap=128, debug=True, debug_short=True)
        assert atomo.payload_status(pay) == (5, 0)
        Us = dbg.layer_short(0, 128).astype(np.float64)
        assert np.abs(Us @ Us.T - np.eye(128)).max() <= 1e-4
    finally:
        atomo.set_eig_params(40, 3e-7)
        atomo.set_eig_mode(1)
        atomo.set_persistent_eig(3)


def test_unbiased_on_gpu(atomo):
    # Lemma 1: mean of many encode+decode passes approaches G; mean #kept atoms approaches s
    import torch
    rng = np.random.default_rng(3)
    G = synth.lowrank_plus_noise(rng, 24, 40, 1.0, noise_rel=0.05)
    t = torch.from_numpy(G).cuda()
    acc = torch.zeros(24, 40, dtype=torch.float64, device="cuda")
    trials, s, kept = 600, 3.0, 0
    for i in range(trials):
        pay, _ = atomo.atomo_encode_spectral([t], s, seed=500 + i, k_cap=24)
        acc += atomo.atomo_decode(pay)[0].double()
        kept += pay.headers()[1][0].k
    U, sig, Vt = np.linalg.svd(G.astype(np.float64), full_matrices=False)
    p = np.minimum(1.0, s * sig / sig.sum())
    assert s <= sig.sum() / sig.max()
    var = np.einsum("i,ai,ib->ab", sig ** 2 * (1 - p) / p, U ** 2, Vt ** 2)
    mean = (acc / trials).cpu().numpy()
    assert np.all(np.abs(mean - G) <= 6 * np.sqrt(var / trials) + 1e-6)
    assert abs(kept / trials - s) <= 6 * np.sqrt(np.sum(p * (1 - p)) / trials)


def test_config2_full(atomo, oracle):
    # the benchmark workload: all 18 ResNet-18-shaped layers in one batched call, s = 2
    mats = synth.c2_resnet18(0)
    before = dict(parity.TALLY)
    _run(atomo, oracle, mats, 2.0, seed=2024, step=1)
    t = parity.TALLY
    print({k: (t[k] - before[k] if k != "worst_err_times_gap" else t[k]) for k in t})
    assert t["masks_identical"] - before["masks_identical"] == len(mats)
    assert t["terms_compared"] - before["terms_compared"] >= len(mats) // 2


def test_config5_shape_properties(atomo):
    # 1024 x 4096 layers (the stress-test shape): the oracle SVD takes minutes there, so the
    # checks are those that hold at any size, evaluated in fp64 -- singular values against a
    # library SVD, kept atoms as singular triplets, the decode kernel against its definition
    import torch
    mats = synth.c5_stress(0, count=2)
    for s in (2.0, 8.0):
        pay, dbg = _encode(atomo, mats, s, seed=77, k_cap=64)
        hdrs = pay.headers()
        outs = atomo.atomo_decode(pay)
        for l, G in enumerate(mats):
            G64 = G.astype(np.float64)
            ref = np.linalg.svd(G64, compute_uv=False)
            h = hdrs[1][l]
            assert h.status == 0
            sig = dbg.layer_sigma(l, 1024)
            assert parity.rel(sig, ref) <= parity.REL_TOL
            arr = pay.layer_arrays(l, hdrs)
            p = dbg.layer_prob(l, 1024)
            assert abs(p.sum() - s) <= 1e-4 * s
            for j in range(arr["k"]):
                u = arr["U"][:, j].astype(np.float64); v = arr["V"][:, j].astype(np.float64)
                sg = float(arr["coef"][j]) * float(p[arr["idx"][j]])
                assert np.linalg.norm(G64.T @ u - sg * v) <= 2e-5 * ref[0]
                assert np.linalg.norm(G64 @ v - sg * u) <= max(2e-5 * ref[0], parity.RESID_GRAM * ref[0] ** 2 / sg)
            own = (arr["U"].astype(np.float64) * arr["coef"].astype(np.float64)) @ arr["V"].astype(np.float64).T
            out = outs[l].cpu().numpy()
            assert (parity.rel(out, own) <= 1e-5) if arr["k"] else (not out.any())
            parity.check_full_basis(G, dbg, l, f"L{l}", orth_tol=2e-3)
        if s == 8.0:
            assert all(h.n_sat >= 1 for h in hdrs[1])          # sum(sigma) ~ 7.5 < 8 sigma_1


@pytest.mark.parametrize("scheme", [3, 1])
def test_config5_full_size(atomo, scheme):
    """Config 5 at its full size (96 layers of 1024 x 4096, 402,653,184 elements) on the default route (the blocked
    tridiagonal reduction, one CTA per layer) and on the Jacobi fallback (more block pairs than the GPU holds CTAs, so
    that eigen-solve runs as a sequence of persistent launches over groups of layers).  Six distinct
    seeded matrices, each used 16 times (generating 96 Haar factors of order 4096 would take minutes on the host);
    every copy is its own layer with its own Philox stream.  Checked: status, singular values against a library SVD
    in fp64, sum(p) = s, kept atoms as singular triplets on sampled layers, the decode against its definition."""
    import torch
    base = synth.c5_stress(0, count=6)
    refs = [np.linalg.svd(G.astype(np.float64), compute_uv=False) for G in base]
    dev = torch.device("cuda:0")
    ts = [torch.from_numpy(base[i % 6]).to(dev).clone() for i in range(96)]
    s = 4.0
    try:
        atomo.set_persistent_eig(scheme)
        pay, dbg = atomo.atomo_encode_spectral(ts, s, seed=91, step=5, k_cap=48, debug=True)
    finally:
        atomo.set_persistent_eig(3)
    assert atomo.last_eig_scheme() == scheme
    hdrs = pay.headers()
    assert [h.status for h in hdrs[1]] == [0] * 96
    outs = atomo.atomo_decode(pay)
    ks = [h.k for h in hdrs[1]]
    assert len(set(ks)) > 1                                   # the copies draw from different Philox streams
    for l in range(96):
        sig = dbg.layer_sigma(l, 1024)
        assert parity.rel(sig, refs[l % 6]) <= parity.REL_TOL
        p = dbg.layer_prob(l, 1024)
        assert abs(p.sum() - s) <= 1e-4 * s
    for l in (0, 17, 40, 63, 95):                             # kept atoms of a few layers, in fp64
        G64 = base[l % 6].astype(np.float64)
        ref = refs[l % 6]
        arr = pay.layer_arrays(l, hdrs)
        p = dbg.layer_prob(l, 1024)
        for j in range(arr["k"]):
            u = arr["U"][:, j].astype(np.float64); v = arr["V"][:, j].astype(np.float64)
            sg = float(arr["coef"][j]) * float(p[arr["idx"][j]])
            assert np.linalg.norm(G64.T @ u - sg * v) <= 2e-5 * ref[0]
            assert np.linalg.norm(G64 @ v - sg * u) <= max(2e-5 * ref[0], parity.RESID_GRAM * ref[0] ** 2 / sg)
        own = (arr["U"].astype(np.float64) * arr["coef"].astype(np.float64)) @ arr["V"].astype(np.float64).T
        out = outs[l].cpu().numpy()
        assert (parity.rel(out, own) <= 1e-5) if arr["k"] else (not out.any())


def test_eigen_routes_agree(atomo, oracle):
    # route 0 (Jacobi on [A | I] with accumulated vectors) is an independent check of route 1
    # (Cholesky factor, Jacobi on its rows): same singular values, probabilities and masks
    L = synth.RESNET18_LAYERS
    mats = synth.c2_resnet18(2, [L[1], L[6], L[10], L[17]])
    try:
        atomo.set_eig_mode(0)
        pay0, dbg0 = _encode(atomo, mats, 2.0, seed=31, step=2)
        _run(atomo, oracle, mats, 2.0, seed=31, step=2)
    finally:
        atomo.set_eig_mode(1)
    pay1, dbg1 = _encode(atomo, mats, 2.0, seed=31, step=2)
    for l, G in enumerate(mats):
        r = min(G.shape)
        assert parity.rel(dbg1.layer_sigma(l, r), dbg0.layer_sigma(l, r)) <= 3e-5
        assert parity.rel(dbg1.layer_prob(l, r), dbg0.layer_prob(l, r)) <= 3e-5


def test_config3_vgg11_properties(atomo):
    # VGG-11-shaped set with two 4096 x 4096 layers, budgets 1, 2, 3.  The oracle SVD would take hours
    # there, so the checks are the ones that hold at any size, in fp64: singular values against a library
    # SVD, sum(p) = s, kept atoms as singular triplets, the decode kernel against its definition, and the
    # small layers against the expected saturation (the 10 x 4096 layer saturates at s = 3)
    import torch
    mats = synth.c3_vgg11(0)
    refs = [np.linalg.svd(G.astype(np.float64), compute_uv=False) for G in mats]
    ts = [torch.from_numpy(G).cuda() for G in mats]
    for s in (1.0, 2.0, 3.0):
        pay, dbg = atomo.atomo_encode_spectral(ts, s, seed=900 + int(s), step=int(s), k_cap=32, debug=True)
        hdrs = pay.headers()
        outs = atomo.atomo_decode(pay)
        assert [h.status for h in hdrs[1]] == [0] * len(mats)
        for l, G in enumerate(mats):
            r = min(G.shape)
            ref = refs[l]
            sig = dbg.layer_sigma(l, r); p = dbg.layer_prob(l, r)
            assert parity.rel(sig, ref) <= parity.REL_TOL, f"L{l}: sigma {parity.rel(sig, ref)}"
            assert abs(p.sum() - min(s, r)) <= 1e-4 * s
            p_ref = np.minimum(1.0, s * ref / ref.sum()) if s <= ref.sum() / ref[0] else None
            if p_ref is not None:
                assert parity.rel(p, p_ref) <= parity.REL_TOL
            arr = pay.layer_arrays(l, hdrs)
            G64 = G.astype(np.float64)
            for j in range(arr["k"]):
                u = arr["U"][:, j].astype(np.float64); v = arr["V"][:, j].astype(np.float64)
                sg = float(arr["coef"][j]) * float(p[arr["idx"][j]])
                r_u = np.linalg.norm(G64.T @ u - sg * v); r_v = np.linalg.norm(G64 @ v - sg * u)
                lo, hi = (r_u, r_v) if G.shape[0] <= G.shape[1] else (r_v, r_u)
                assert lo <= 2e-5 * ref[0]
                assert hi <= max(2e-5 * ref[0], parity.RESID_GRAM * ref[0] ** 2 / sg)
            own = (arr["U"].astype(np.float64) * arr["coef"].astype(np.float64)) @ arr["V"].astype(np.float64).T
            out = outs[l].cpu().numpy()
            assert (parity.rel(out, own) <= 1e-5) if arr["k"] else (not out.any())
        if s == 3.0:
            assert hdrs[1][10].n_sat >= 1          # 10 x 4096: sum(sigma) ~ 2.93 sigma_1 < 3 sigma_1


def test_sigma_refinement_all_layers(atomo, oracle):
    # with the projection-norm refinement on for every layer the parity protocol still holds; with the
    # fp32 FMA Gram kernel the probabilities then land within 2e-6 of the oracle's and sigma within
    # 1e-6 sigma_1 (the Gram route alone is about 10x further away); with the tensor-core Gram kernel,
    # whose tail vectors are a little less sharp, within 1e-5
    L = synth.RESNET18_LAYERS
    mats = synth.c2_resnet18(1, [L[1], L[6], L[10], L[14], L[17]])
    atomo.set_sigma_refinement(0)
    try:
        for tensor_cores, p_bar, s_bar in ((False, 2e-6, 1e-6), (True, 1e-5, 5e-6)):
            atomo.set_gram_path(tensor_cores)
            pay, hdrs, encs = _run(atomo, oracle, mats, 2.0, seed=77, step=3)
            pay, dbg = _encode(atomo, mats, 2.0, seed=77, step=3)
            for l, G in enumerate(mats):
                r = min(G.shape)
                assert np.abs(dbg.layer_prob(l, r) - encs[l]["p"]).max() <= p_bar
                assert np.abs(dbg.layer_sigma(l, r) - encs[l]["sigma"]).max() <= s_bar * encs[l]["sigma"][0]
    finally:
        atomo.set_sigma_refinement(2048)
        atomo.set_gram_path(True)


def test_gram_paths_agree(atomo, oracle):
    # the fp32 FMA Gram kernel is an independent check of the tensor-core one (TF32 hi/lo split)
    L = synth.RESNET18_LAYERS
    mats = synth.c2_resnet18(3, [L[0], L[2], L[9], L[13], L[17]])
    try:
        atomo.set_gram_path(False)
        _run(atomo, oracle, mats, 2.0, seed=41, step=6)
        pay0, dbg0 = _encode(atomo, mats, 2.0, seed=41, step=6)
    finally:
        atomo.set_gram_path(True)
    pay1, dbg1 = _encode(atomo, mats, 2.0, seed=41, step=6)
    for l, G in enumerate(mats):
        r = min(G.shape)
        assert parity.rel(dbg1.layer_sigma(l, r), dbg0.layer_sigma(l, r)) <= 3e-5
        assert np.array_equal(dbg1.layer_mask(l, r), dbg0.layer_mask(l, r))
