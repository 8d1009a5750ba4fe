"""GPU parity: entry-wise ATOMO through the C ABI vs the fp64 oracle (bit-exact masks/indices)."""
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


def _run(atomo, oracle, vecs, s, seed, step=0, k_cap=None, offset=0):
    import torch
    dev = torch.device("cuda:0")
    ts = []
    for g in vecs:
        buf = torch.zeros(g.size + offset, dtype=torch.float32, device=dev)
        buf[offset:] = torch.from_numpy(g).to(dev)
        ts.append(buf[offset:])
    if k_cap is None:
        k_cap = max(g.size for g in vecs)
    pay, dbg = atomo.atomo_encode_entrywise(ts, s, seed, step=step, k_cap=k_cap, debug=True)
    hdrs = pay.headers()
    outs = atomo.atomo_decode(pay)
    report = []
    for l, g in enumerate(vecs):
        arr = pay.layer_arrays(l, hdrs)
        same, enc = parity.check_entrywise(atomo, oracle, g, ts[l], s, seed, step, arr, hdrs[1][l], dbg, l, report,
                                           f"vec{l}[n={g.size},s={s:g}]")
        out = outs[l].cpu().numpy()
        # decode kernel: exactly the payload's values at the payload's indices, zeros elsewhere
        want = np.zeros(g.size, dtype=np.float32)
        want[arr["idx"].astype(np.int64)] = arr["val"]
        assert np.array_equal(out, want)
        if same:
            ref = oracle.decode_entrywise(g.size, enc["idx"], enc["val"])
            assert parity.rel(out, ref) <= parity.REL_TOL if enc["idx"].size else not out.any()
    print("\n".join(report))
    # Without the probabilities asked for, the one-kernel form takes the keep decisions on the candidate list of its
    # first pass wherever that list is complete: the same masks and payload arrays have to come out.
    pay2, dbg2 = atomo.atomo_encode_entrywise(ts, s, seed, step=step, k_cap=k_cap, debug="mask")
    hdrs2 = pay2.headers()
    assert torch.equal(dbg2.mask_words, dbg.mask_words), "mask words differ when the probabilities are not asked for"
    for l in range(len(vecs)):
        h, h2 = hdrs[1][l], hdrs2[1][l]
        assert (h.status, h.k, h.n_sat, h.c, h.l1) == (h2.status, h2.k, h2.n_sat, h2.c, h2.l1)
        a, a2 = pay.layer_arrays(l, hdrs), pay2.layer_arrays(l, hdrs2)
        assert np.array_equal(a["idx"], a2["idx"]) and np.array_equal(a["val"], a2["val"])
    return pay, hdrs


def test_config1_entrywise(atomo, oracle):
    _run(atomo, oracle, [synth.c1_entrywise(0)], 64.0, seed=1, step=3)


def test_qsgd_and_terngrad_budgets(atomo, oracle):
    # Section 4: s = ||g||_1/||g||_2 and ||g||_1/||g||_inf; kept values are +-||g||_q
    g = synth.c1_entrywise(1)
    l1 = float(np.abs(g.astype(np.float64)).sum())
    for nq in (float(np.linalg.norm(g.astype(np.float64))), float(np.abs(g).max())):
        pay, hdrs = _run(atomo, oracle, [g], l1 / nq, seed=2)
        arr = pay.layer_arrays(0, hdrs)
        np.testing.assert_allclose(np.abs(arr["val"]), nq, rtol=2e-6)


@pytest.mark.parametrize("s", [2000.0, 4095.5, 5000.0])
def test_unbalanced_budgets_saturate(atomo, oracle, s):
    pay, hdrs = _run(atomo, oracle, [synth.c1_entrywise(1)], s, seed=5)
    assert hdrs[1][0].n_sat > 0


@pytest.mark.parametrize("n", [1, 3, 5, 31, 4095, 4096, 4097, 12289, 1_000_003])
def test_ragged_lengths(atomo, oracle, n):
    g = synth.c4_entrywise(3, n=n)
    _run(atomo, oracle, [g], max(0.5, n / 100.0), seed=9, step=17)


def test_batch_and_layer_index(atomo, oracle):
    vecs = [synth.c4_entrywise(1, n=5000), synth.c1_entrywise(2), synth.c4_entrywise(2, n=70001)]
    _run(atomo, oracle, vecs, 40.0, seed=0xDEADBEEFCAFE, step=2 ** 31 + 5)


def test_unaligned_pointer(atomo, oracle):
    _run(atomo, oracle, [synth.c4_entrywise(4, n=10007)], 55.5, seed=4, offset=1)


def test_zeros(atomo, oracle):
    g = synth.c1_entrywise(3).copy()
    g[::3] = 0.0
    _run(atomo, oracle, [g], 3000.0, seed=8)      # s > number of non-zero atoms: all of them kept
    pay, hdrs = _run(atomo, oracle, [np.zeros(5000, dtype=np.float32)], 10.0, seed=8)
    assert hdrs[1][0].k == 0


def test_deterministic(atomo):
    import torch
    g = torch.from_numpy(synth.c4_entrywise(5, n=300_001)).cuda()
    p1, _ = atomo.atomo_encode_entrywise([g], 3000.0, seed=3, k_cap=5000)
    p2, _ = atomo.atomo_encode_entrywise([g], 3000.0, seed=3, k_cap=5000)
    h = p1.headers()[1][0]
    a1, a2 = p1.layer_arrays(0), p2.layer_arrays(0)
    assert h.k > 0 and np.array_equal(a1["idx"], a2["idx"]) and np.array_equal(a1["val"], a2["val"])
    p3, _ = atomo.atomo_encode_entrywise([g], 3000.0, seed=4, k_cap=5000)
    assert not np.array_equal(p3.layer_arrays(0)["idx"], a1["idx"])


def test_device_side_errors(atomo):
    import torch
    g = synth.c1_entrywise(0).copy()
    t = torch.from_numpy(g).cuda()
    # more kept atoms than k_cap: status, k = 0, decode gives zeros (never a silent truncation)
    pay, _ = atomo.atomo_encode_entrywise([t], 64.0, seed=1, k_cap=10)
    assert atomo.payload_status(pay) == (3, 0)
    assert pay.headers()[1][0].k == 0 and not atomo.atomo_decode(pay)[0].any()
    g[7] = np.nan
    pay, _ = atomo.atomo_encode_entrywise([torch.from_numpy(g).cuda()], 64.0, seed=1, k_cap=4096)
    assert atomo.payload_status(pay) == (4, 0) and pay.headers()[1][0].k == 0
    g[7] = np.inf
    pay, _ = atomo.atomo_encode_entrywise([torch.from_numpy(g).cuda()], 64.0, seed=1, k_cap=4096)
    assert atomo.payload_status(pay)[0] == 4


def test_host_side_errors(atomo):
    import torch
    from paper_1806_04090_b200 import api
    t = torch.ones(100, device="cuda")
    for bad in (0.0, -2.0, float("nan"), float("inf")):
        with pytest.raises(api.AtomoError) as e:
            atomo.atomo_encode_entrywise([t], bad, seed=1)
        assert e.value.code == 2
    with pytest.raises(api.AtomoError) as e:
        atomo.atomo_encode_entrywise([t], 5.0, seed=1, k_cap=50, payload=torch.empty(64, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 3
    # decode with the wrong shape: payload status, zeros written
    pay, _ = atomo.atomo_encode_entrywise([t], 5.0, seed=1, k_cap=100)
    pay.shapes = [(1, 99)]
    out = atomo.atomo_decode(pay)[0]
    assert not out.any() and atomo.payload_status(pay)[0] == 8


def test_unbiased_on_gpu(atomo):
    # Lemma 1 at a size the oracle never sees: the mean of many decodes approaches g
    import torch
    g = torch.from_numpy(synth.c4_entrywise(6, n=20000)).cuda()
    acc = torch.zeros_like(g, dtype=torch.float64)
    trials = 400
    s = 2000.0
    for t in range(trials):
        pay, _ = atomo.atomo_encode_entrywise([g], s, seed=100 + t, k_cap=4000)
        acc += atomo.atomo_decode(pay)[0].double()
    mean = (acc / trials).cpu().numpy()
    g64 = g.double().cpu().numpy()
    p = np.minimum(1.0, np.abs(g64) * s / np.abs(g64).sum())       # balanced here
    sd = np.sqrt(g64 ** 2 * (1 - p) / np.maximum(p, 1e-300) / trials)
    assert np.all(np.abs(mean - g64) <= 6 * sd + 1e-12)
    assert abs(np.sum(mean) - np.sum(g64)) <= 6 * np.sqrt(np.sum(sd ** 2))


@pytest.mark.parametrize("frac", [0.001, 0.01, 0.1])
def test_config4_full_size(atomo, oracle, frac):
    # 25.6M Laplace(0, 1e-3) entries, budgets 0.1 %, 1 %, 10 % of the length, in the bench's launch configuration
    g = synth.c4_entrywise(0)
    _run(atomo, oracle, [g], frac * g.size, seed=7, step=1, k_cap=int(frac * g.size * 1.05) + 1000)


def test_lq_budget_front_end(atomo, oracle):
    """atomo_lq_budget against the plain definition, and the budgets fed back into the encoder (Section 4)."""
    import torch
    rng = np.random.default_rng(31)
    vecs = [synth.c1_entrywise(2), (rng.laplace(0.0, 1e-3, 1_000_003)).astype(np.float32), np.zeros(100, dtype=np.float32)]
    ts = [torch.from_numpy(v).cuda() for v in vecs]
    for q in (1.0, 2.0, 3.5, float("inf")):
        got = atomo.atomo_lq_budget(ts, q)
        for v, s_gpu in zip(vecs, got):
            want = oracle.lq_budget(v, q)
            assert s_gpu == pytest.approx(want, rel=1e-12, abs=0.0), (q, s_gpu, want)
    # QSGD budget: kept unsaturated values are +-||g||_2 (already covered with host-computed budgets; here end to end)
    g = vecs[0]
    s2 = atomo.atomo_lq_budget(ts[:1], 2.0)[0]
    pay, _ = atomo.atomo_encode_entrywise(ts[:1], s2, seed=3, k_cap=g.size)
    arr = pay.layer_arrays(0)
    assert pay.headers()[1][0].n_sat == 0
    np.testing.assert_allclose(np.abs(arr["val"]), np.linalg.norm(g.astype(np.float64)), rtol=1e-6)
    bad = torch.tensor([1.0, float("nan"), 2.0], device="cuda")
    assert np.isnan(atomo.atomo_lq_budget([bad], 2.0)[0])
    with pytest.raises(Exception):
        atomo.atomo_lq_budget(ts[:1], 0.5)


def test_which_chunks_decide_on_their_list(atomo):
    """The one-kernel form counts the chunks that took their keep decisions on the candidate list of the first pass:
    all of them on an s-balanced vector with a small budget; none when the probabilities are asked for, when the
    vector is not s-balanced or the budget is large (the host then launches the form without the list) or in the
    two-kernel form; some where a chunk's own estimate of sum |g| is off (half the vector zero: the chunks of the zero
    half hold no candidate and confirm trivially, the others overestimate sum |g| twofold and read their part again)."""
    import torch
    rng = np.random.default_rng(78)
    big = rng.laplace(0.0, 1e-3, 3_000_017).astype(np.float32)
    spiky = big.copy(); spiky[rng.choice(spiky.size, 300, replace=False)] *= 1.0e4
    half = big.copy(); half[: half.size // 2] = 0.0
    t = lambda g: [torch.from_numpy(g).cuda()]
    s = 0.01 * big.size
    try:
        atomo.atomo_encode_entrywise(t(big), s, seed=5, k_cap=int(1.2 * s) + 2000)
        got, chunks = atomo.entrywise_list_chunks(0)
        assert chunks > 100 and got == chunks
        atomo.atomo_encode_entrywise(t(big), s, seed=5, k_cap=int(1.2 * s) + 2000, debug=True)
        got_p, chunks_p = atomo.entrywise_list_chunks(0)                  # the form without the list: more, smaller CTAs
        assert got_p == 0 and chunks_p > 100
        atomo.atomo_encode_entrywise(t(spiky), 5000.0, seed=5, k_cap=8000)
        assert atomo.entrywise_list_chunks(0) == (0, chunks)
        # chunks of two tiles: a thread still expects few candidates at 4 % of the length, far too many at 12 %
        atomo.atomo_encode_entrywise(t(big), 4.0 * s, seed=5, k_cap=int(4.8 * s) + 2000)
        assert atomo.entrywise_list_chunks(0) == (chunks, chunks)
        atomo.atomo_encode_entrywise(t(big), 12.0 * s, seed=5, k_cap=int(14.0 * s) + 2000)
        got12, chunks12 = atomo.entrywise_list_chunks(0)
        assert got12 == 0 and chunks12 > 100
        atomo.atomo_encode_entrywise(t(half), s, seed=5, k_cap=int(1.2 * s) + 2000)
        got_h, chunks_h = atomo.entrywise_list_chunks(0)
        assert chunks_h == chunks and 0.3 * chunks < got_h < 0.7 * chunks
        atomo.set_entrywise_launch(1)
        atomo.atomo_encode_entrywise(t(big), s, seed=5, k_cap=int(1.2 * s) + 2000)
        assert atomo.entrywise_list_chunks(0) == (0, 0)
    finally:
        atomo.set_entrywise_launch(0)


@pytest.mark.parametrize("compact", [False, True])
def test_launch_forms_agree(atomo, compact):
    """The one-kernel form (solve, grid barrier, sample and pack in one cooperative launch) and the two-kernel form
    (solve kernel, then sample / pack with chunks handed out by ticket) cut the vector into different chunks on a
    different number of CTAs: mask words, kept indices, values and decoded gradients have to be identical all the
    same.  (sum |g| is added up in short fp32 runs and then chunk by chunk in fp64, so it depends on the cut at the
    1e-8 level: it is compared to 1e-7.  The weight c = T / (s - n_s) and the scale of the probabilities are its
    fp32 roundings; where they come out equal -- they do for these inputs -- everything else has to be identical.)
    The one-kernel form is run three ways: deciding on the candidate list of its first pass (the default), without the
    list (launch form 2), and with the probabilities asked for, which switches the list off as well."""
    import torch
    from paper_1806_04090_b200 import api
    rng = np.random.default_rng(77)
    big = rng.laplace(0.0, 1e-3, 3_000_017).astype(np.float32)
    spiky = rng.laplace(0.0, 1e-3, 700_001).astype(np.float32)
    spiky[rng.choice(spiky.size, 300, replace=False)] *= 1.0e4          # not s-balanced: saturated atoms
    # inputs on which a chunk's own estimate of sum |g| is wrong in either direction, so that some chunks of the
    # one-kernel form decide on their candidate list and others read their part a second time: half the vector zero,
    # a scale that grows a hundredfold along the vector, and zero first tiles followed by data
    half = big.copy(); half[: half.size // 2] = 0.0
    ramp = (big * np.linspace(0.05, 5.0, big.size, dtype=np.float32)).astype(np.float32)
    holes = big.copy(); holes.reshape(-1)[: (holes.size // 8192) * 8192].reshape(-1, 8192)[:, :4096] = 0.0
    cases = [([big], 0.01 * big.size), ([spiky], 5000.0), ([big[:4097], spiky[:123], big[:40960]], 64.0),
             ([half], 0.01 * big.size), ([ramp], 0.01 * big.size), ([holes], 0.002 * big.size), ([big], 0.04 * big.size)]
    try:
        for vecs, s in cases:
            ts = [torch.from_numpy(g).cuda() for g in vecs]
            k_cap = int(1.2 * s) + 2000
            got = []
            # (launch form, debug outputs): the one-kernel form with the candidate list first (asking for the
            # probabilities switches the list off), then the two-kernel form and the one-kernel form without the list
            for form, debug in ((0, "mask"), (1, True), (2, True), (0, True)):
                atomo.set_entrywise_launch(form)
                atomo.set_entrywise_format(api.EW_COMPACT if compact else api.EW_EXPLICIT, 1000 if compact else 0)
                pay, dbg = atomo.atomo_encode_entrywise(ts, s, seed=5, step=3, k_cap=k_cap, debug=debug)
                outs = atomo.atomo_decode(pay)
                torch.cuda.synchronize()
                hdrs = pay.headers()
                assert max(h.status for h in hdrs[1]) == 0
                got.append((hdrs[1], [pay.layer_arrays(l, hdrs) for l in range(len(vecs))], dbg.mask_words.clone(),
                            [o.clone() for o in outs]))
            for other in got[1:]:
                for l in range(len(vecs)):
                    h0, h1 = got[0][0][l], other[0][l]
                    assert abs(h0.l1 - h1.l1) <= 1e-7 * abs(h0.l1)
                    assert h0.c == h1.c, "the fp32 weight differs between the launch forms: choose other test inputs"
                assert torch.equal(got[0][2], other[2]), "mask words differ between the launch forms"
                for l in range(len(vecs)):
                    h0, h1 = got[0][0][l], other[0][l]
                    assert (h0.k, h0.n_sat, h0.sweeps) == (h1.k, h1.n_sat, h1.sweeps)
                    a0, a1 = got[0][1][l], other[1][l]
                    assert np.array_equal(a0["idx"], a1["idx"]) and np.array_equal(a0["val"], a1["val"])
                    assert torch.equal(got[0][3][l], other[3][l])
    finally:
        atomo.set_entrywise_launch(False)
        atomo.set_entrywise_format(api.EW_EXPLICIT, 0)
