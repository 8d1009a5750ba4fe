"""GPU parity of the blocked tridiagonal route (short sides above 512) against the fp64 oracle, at sizes the oracle
finishes in seconds, and the properties of that route: the payload does not depend on the number of CTAs per
layer, small and large layers share one call."""
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


def _mat(seed, m, n, decay=1.0, noise=0.01):
    return synth.lowrank_plus_noise(np.random.default_rng([77, seed, m, n]), m, n, decay, noise_rel=noise)


def _encode(atomo, mats, s, seed, step=0, k_cap=64):
    import torch
    ts = [torch.from_numpy(G).cuda() for G in mats]
    return atomo.atomo_encode_spectral(ts, s, seed, step=step, k_cap=k_cap, debug=True)


def _against_oracle(atomo, oracle, mats, s, seed, step):
    pay, dbg = _encode(atomo, mats, s, seed, step)
    assert atomo.last_eig_scheme() == 3
    hdrs = pay.headers()
    outs = atomo.atomo_decode(pay)
    encs = parity.oracle_spectral_batch(oracle, mats, s, seed, step)
    report = []
    for l, G in enumerate(mats):
        r = min(G.shape)
        arr = pay.layer_arrays(l, hdrs)
        out = outs[l].cpu().numpy().astype(np.float64)
        parity.check_spectral_layer(oracle, G, encs[l], hdrs[1][l], arr, dbg, l, out, report, f"L{l}{G.shape}",
                                    gap_min=parity.gap_min_for(r, atomo.last_eig_scheme()))
        dp = float(np.abs(dbg.layer_prob(l, r) - encs[l]["p"]).max())
        report.append(f"L{l}{G.shape}: max |p - p_oracle| = {dp:.2e}")
        assert dp <= 2e-6
        U = arr["U"].astype(np.float64) if G.shape[0] <= G.shape[1] else arr["V"].astype(np.float64)
        if arr["k"]:
            assert np.abs(U.T @ U - np.eye(arr["k"])).max() <= 2e-5     # kept short-side vectors orthonormal
    print("\n".join(report))


# ctas = 0: clusters sized by the batch (the cluster kernel); ctas = 1: one CTA per layer (the triangle-only kernel that
# large batches such as config 5 take)
@pytest.mark.parametrize("ctas", [0, 1])
@pytest.mark.parametrize("shape", [(513, 700), (600, 1500), (900, 640), (1000, 1100), (1023, 1030)])
def test_ragged_short_sides_against_oracle(atomo, oracle, shape, ctas):
    try:
        atomo.set_tridiag_ctas(ctas)
        _against_oracle(atomo, oracle, [_mat(1, *shape)], 3.0, seed=41, step=2)
    finally:
        atomo.set_tridiag_ctas(0)


@pytest.mark.parametrize("ctas", [0, 1])
def test_mixed_batch_against_oracle(atomo, oracle, ctas):
    # small layers (register-resident reduction) and large ones (blocked reduction) in one call
    mats = [_mat(2, 64, 576), _mat(3, 640, 800), _mat(4, 256, 1152), _mat(5, 10, 600), _mat(6, 770, 771)]
    try:
        atomo.set_tridiag_ctas(ctas)
        _against_oracle(atomo, oracle, mats, 2.0, seed=43, step=1)
    finally:
        atomo.set_tridiag_ctas(0)


def test_payload_independent_of_ctas_per_layer(atomo):
    """The cluster kernel orders every sum independently of the number of CTAs per layer: 2, 4, 8 and 16 CTAs give the
    same payload bit for bit (a second launch geometry of the same arithmetic).  One CTA per layer runs another
    kernel (triangle-only products, panels of 16): the same atoms are kept and the values agree to rounding."""
    mats = [_mat(7, 1024, 2048), _mat(8, 777, 1300)]
    got = {}
    try:
        for ctas in (1, 2, 4, 8, 16):
            atomo.set_tridiag_ctas(ctas)
            pay, dbg = _encode(atomo, mats, 4.0, seed=5, step=9)
            hdrs = pay.headers()
            assert [h.status for h in hdrs[1]] == [0, 0]
            arrs = [pay.layer_arrays(l, hdrs) for l in range(2)]
            got[ctas] = [dbg.sigma.cpu().numpy(), dbg.prob.cpu().numpy(), dbg.mask_words.cpu().numpy()] + \
                        [np.array(a[key]) for a in arrs for key in ("idx", "coef", "U", "V")]
    finally:
        atomo.set_tridiag_ctas(0)
    for ctas in (4, 8, 16):
        for a, b in zip(got[2], got[ctas]):
            assert a.shape == b.shape and np.array_equal(a.view(np.uint32) if a.dtype == np.float32 else a,
                                                         b.view(np.uint32) if b.dtype == np.float32 else b)
    one, two = got[1], got[2]
    # sigma: the tail values (1e-3 sigma_1) differ by about 1e-7 sigma_1 between two fp32 summation orders
    assert parity.rel(one[0], two[0]) <= 5e-6 and np.abs(one[1] - two[1]).max() <= 1e-6
    assert np.array_equal(one[2], two[2])                                                     # masks
    for a, b in zip(one[3:], two[3:]):
        assert a.shape == b.shape
        if a.dtype == np.float32 and a.ndim == 2 and a.size:     # vectors: the same up to sign-free rounding
            assert np.abs(np.abs(np.sum(a * b, axis=0)) - 1.0).max() <= 1e-4
        elif a.dtype == np.float32:
            assert parity.rel(a, b) <= 1e-5
        else:
            assert np.array_equal(a, b)


def test_saturated_and_rank_deficient_large_layers(atomo, oracle):
    rng = np.random.default_rng(9)
    # rank 3 plus nothing: 597 zero singular values.  With a budget above the rank the three atoms have p = 1 and the
    # decode returns G.  (The eigenvalues of an fp32 Gram matrix resolve singular values only down to about 1e-4 of
    # the largest: atoms below that get noise-level probabilities instead of exactly 0, and one of them may be
    # drawn; its weight is the norm of its back-projection, which is at rounding level.)
    u = np.linalg.qr(rng.standard_normal((600, 3)))[0]
    v = np.linalg.qr(rng.standard_normal((900, 3)))[0]
    G = ((u * np.array([3.0, 2.0, 1.0])) @ v.T).astype(np.float32)
    pay, dbg = _encode(atomo, [G], 5.0, seed=1)
    hdrs = pay.headers()
    assert hdrs[1][0].status == 0 and hdrs[1][0].k >= 3 and hdrs[1][0].n_sat == 3
    assert list(pay.layer_arrays(0, hdrs)["idx"][:3]) == [0, 1, 2]
    out = atomo.atomo_decode(pay)[0].cpu().numpy()
    assert parity.rel(out, G) <= 1e-5
    sig = dbg.layer_sigma(0, 600)
    assert np.allclose(sig[:3], [3, 2, 1], rtol=1e-5) and np.all(sig[3:] <= 1e-3)
    # zero matrix and a NaN: status words, nothing kept
    Z = np.zeros((520, 530), dtype=np.float32)
    N = _mat(10, 530, 540); N[5, 7] = np.nan
    pay, dbg = _encode(atomo, [Z, N], 2.0, seed=1)
    hdrs = pay.headers()
    assert hdrs[1][0].status == 0 and hdrs[1][0].k == 0
    assert hdrs[1][1].status == 4 and hdrs[1][1].k == 0
    outs = atomo.atomo_decode(pay)
    assert not outs[0].any() and not outs[1].any()


def test_large_layers_alone_in_a_fresh_process():
    """A batch that holds nothing but layers above a short side of 3000 (the eigenvalue kernel then needs more than
    the default 48 KB of shared memory) in a process that has encoded nothing else before: the shared-memory opt-ins
    of every kernel on the way must not depend on another route having been configured first."""
    import subprocess
    import sys
    code = (
        "import numpy as np, torch\n"
        "from paper_1806_04090_b200 import api, synth\n"
        "a = api.Atomo(0)\n"
        "G = synth.torch_lowrank_plus_noise(3100, 3200, 1.0, 5, torch.device('cuda:0'), noise_rel=0.01)\n"
        "pay, dbg = a.atomo_encode_spectral([G], 2.0, seed=3, step=1, k_cap=16, debug=True)\n"
        "h = pay.headers()[1][0]\n"
        "assert h.status == 0 and a.last_eig_scheme() == 3, (h.status, a.last_eig_scheme())\n"
        "sig = dbg.layer_sigma(0, 3100)\n"
        "ref = torch.linalg.svdvals(G.double()).cpu().numpy()\n"
        "assert np.linalg.norm(sig - ref) <= 1e-4 * np.linalg.norm(ref)\n"
        "out = a.atomo_decode(pay)[0]\n"
        "assert torch.isfinite(out).all()\n"
        "print('ok', int(h.k))\n")
    res = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0 and res.stdout.strip().startswith("ok"), res.stdout + res.stderr
