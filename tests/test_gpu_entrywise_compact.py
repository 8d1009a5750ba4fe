"""GPU parity of the compact entry-wise payload (Section 4's ternary form: a kept atom with p < 1 has the value
sign(g_i) c, so the payload carries a 16-bit entry per such atom, one scalar c, and explicit values only for the
atoms with p = 1).  The kept set, the values and the decoded gradient must equal the explicit format's bit for bit,
and both must match the fp64 oracle."""
import numpy as np
import pytest

from paper_1806_04090_b200 import synth
from tests import parity
from tests.test_gpu_entrywise import _run

pytestmark = pytest.mark.gpu


@pytest.fixture()
def pair():
    """(explicit context, compact context); the compact one starts with room for every atom to saturate."""
    import torch
    from paper_1806_04090_b200 import api
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    a, c = api.Atomo(0), api.Atomo(0)
    c.set_entrywise_format(api.EW_COMPACT, sat_cap=2 ** 31)
    yield a, c
    a.close(); c.close()


def _both(pair, vecs, s, seed, step=0, k_cap=None, sat_cap=None):
    """Encode with both formats; the expanded payloads, the masks and the decodes must agree exactly."""
    import torch
    from paper_1806_04090_b200 import api
    a, c = pair
    if sat_cap is not None:
        c.set_entrywise_format(api.EW_COMPACT, sat_cap=sat_cap)
    ts = [torch.from_numpy(g).cuda() for g in vecs]
    if k_cap is None:
        k_cap = max(g.size for g in vecs)
    pe, de = a.atomo_encode_entrywise(ts, s, seed, step=step, k_cap=k_cap, debug=True)
    pc, dc = c.atomo_encode_entrywise(ts, s, seed, step=step, k_cap=k_cap, debug=True)
    assert pc.ew_format == api.EW_COMPACT and pe.ew_format == api.EW_EXPLICIT
    assert a.payload_status(pe)[0] == 0 and c.payload_status(pc)[0] == 0
    he, hc = pe.headers(), pc.headers()
    assert hc[0].ew_format == api.EW_COMPACT and he[0].ew_format == api.EW_EXPLICIT
    assert torch.equal(de.mask_words, dc.mask_words) and torch.equal(de.prob, dc.prob)
    oe, oc = a.atomo_decode(pe), c.atomo_decode(pc)
    for l in range(len(vecs)):
        ae, ac = pe.layer_arrays(l, he), pc.layer_arrays(l, hc)
        assert he[1][l].k == hc[1][l].k and he[1][l].c == hc[1][l].c
        assert hc[1][l].n_sat == he[1][l].n_sat                  # every saturated atom is kept
        assert np.array_equal(ae["idx"], ac["idx"])
        assert np.array_equal(ae["val"].view(np.uint32), ac["val"].view(np.uint32))
        # the offset table counts the entries (kept atoms with p < 1) before each tile
        sat = np.abs(ae["val"]) != np.float32(hc[1][l].c) if hc[1][l].n_sat else np.zeros(ae["k"], dtype=bool)
        if int(sat.sum()) == hc[1][l].n_sat:                     # (a saturated |g| could equal c exactly)
            tiles = ae["idx"][~sat].astype(np.int64) // 4096
            n_tiles = (vecs[l].size + 4095) // 4096
            want = np.concatenate([[0], np.cumsum(np.bincount(tiles, minlength=n_tiles))])
            assert np.array_equal(ac["table"], want)
        assert torch.equal(oe[l], oc[l])
    return pe, pc


def test_compact_matches_oracle_and_explicit(pair, oracle):
    g = synth.c1_entrywise(0)
    _run(pair[1], oracle, [g], 64.0, seed=1, step=3)
    _both(pair, [g], 64.0, seed=1, step=3)


def test_compact_l_q_budgets_need_no_saturated_list(pair, oracle):
    # Section 4: at s = ||g||_1 / ||g||_q every vector is s-balanced, so sat_cap = 0 is enough, and every kept
    # value is +-||g||_q
    from paper_1806_04090_b200 import api
    g = synth.c1_entrywise(1)
    l1 = float(np.abs(g.astype(np.float64)).sum())
    pair[1].set_entrywise_format(api.EW_COMPACT, sat_cap=0)
    for nq in (float(np.linalg.norm(g.astype(np.float64))), float(np.abs(g).max())):
        pay, hdrs = _run(pair[1], oracle, [g], l1 / nq, seed=2)
        assert hdrs[1][0].n_sat == 0
        np.testing.assert_allclose(np.abs(pay.layer_arrays(0, hdrs)["val"]), nq, rtol=2e-6)
        _both(pair, [g], l1 / nq, seed=2)


@pytest.mark.parametrize("s", [2000.0, 4095.5, 5000.0])
def test_compact_saturated_atoms(pair, oracle, s):
    g = synth.c1_entrywise(1)
    pay, hdrs = _run(pair[1], oracle, [g], s, seed=5)
    assert hdrs[1][0].n_sat > 0
    _both(pair, [g], s, seed=5)


@pytest.mark.parametrize("n", [1, 3, 5, 31, 4095, 4096, 4097, 12289, 1_000_003])
def test_compact_ragged_lengths(pair, oracle, n):
    g = synth.c4_entrywise(3, n=n)
    _run(pair[1], oracle, [g], max(0.5, n / 100.0), seed=9, step=17)
    _both(pair, [g], max(0.5, n / 100.0), seed=9, step=17)


def test_compact_batch_unaligned_and_zeros(pair, oracle):
    vecs = [synth.c4_entrywise(1, n=5000), synth.c1_entrywise(2), synth.c4_entrywise(2, n=70001)]
    _run(pair[1], oracle, vecs, 40.0, seed=0xDEADBEEFCAFE, step=2 ** 31 + 5)
    _both(pair, vecs, 40.0, seed=0xDEADBEEFCAFE, step=2 ** 31 + 5)
    _run(pair[1], oracle, [synth.c4_entrywise(4, n=10007)], 55.5, seed=4, offset=1)
    g = synth.c1_entrywise(3).copy()
    g[::3] = 0.0
    _run(pair[1], oracle, [g], 3000.0, seed=8)            # s > number of non-zero atoms: all kept, all saturated
    _both(pair, [g], 3000.0, seed=8)
    pay, hdrs = _run(pair[1], oracle, [np.zeros(5000, dtype=np.float32)], 10.0, seed=8)
    assert hdrs[1][0].k == 0


@pytest.mark.parametrize("frac", [0.001, 0.1])
def test_compact_config4_full_size(pair, oracle, frac):
    # 25.6M Laplace entries in the bench's launch configuration; a heavy-tailed copy below forces saturation
    g = synth.c4_entrywise(0)
    k_cap = int(frac * g.size * 1.05) + 1000
    _run(pair[1], oracle, [g], frac * g.size, seed=7, step=1, k_cap=k_cap)
    _both(pair, [g], frac * g.size, seed=7, step=1, k_cap=k_cap)


def test_compact_full_size_with_saturation(pair, oracle):
    g = synth.c4_entrywise(0).copy()
    rng = np.random.default_rng(77)
    big = rng.choice(g.size, 20000, replace=False)        # spread over many chunks and tiles
    g[big] *= 1.0e4
    s = 0.01 * g.size
    k_cap = int(s * 1.05) + 1000
    pay, hdrs = _run(pair[1], oracle, [g], s, seed=11, k_cap=k_cap)
    assert hdrs[1][0].n_sat > 1000
    _both(pair, [g], s, seed=11, k_cap=k_cap, sat_cap=int(hdrs[1][0].n_sat))     # an exactly full saturated list


def test_compact_more_chunks_than_one_wave(pair):
    # 100M elements: more chunks of 32 tiles than CTAs resident at once, so late chunks start after early ones ended
    rng = np.random.default_rng(5)
    g = rng.laplace(0.0, 1e-3, 100_000_003).astype(np.float32)
    g[rng.choice(g.size, 3000, replace=False)] *= 1.0e4
    pe, pc = _both(pair, [g], 50_000.0, seed=21, k_cap=60_000, sat_cap=4000)
    h = pc.headers()[1][0]
    assert 0 < h.n_sat <= 3000 and abs(int(h.k) - 50_000) < 2000


def test_compact_capacity_errors(pair):
    import torch
    from paper_1806_04090_b200 import api
    a, c = pair
    g = synth.c1_entrywise(1)
    t = torch.from_numpy(g).cuda()
    # saturated list too short: status, k = 0, zeros decoded (never a silent truncation)
    c.set_entrywise_format(api.EW_COMPACT, sat_cap=8)
    pay, _ = c.atomo_encode_entrywise([t], 4095.5, seed=5, k_cap=4096)
    assert c.payload_status(pay) == (3, 0)
    h = pay.headers()[1][0]
    assert h.k == 0 and h.n_sat == 0 and not c.atomo_decode(pay)[0].any()
    # entry list too short
    c.set_entrywise_format(api.EW_COMPACT, sat_cap=4096)
    pay, _ = c.atomo_encode_entrywise([t], 64.0, seed=1, k_cap=10)
    assert c.payload_status(pay) == (3, 0) and not c.atomo_decode(pay)[0].any()
    # the same budget fits once the capacities do
    pay, _ = c.atomo_encode_entrywise([t], 4095.5, seed=5, k_cap=4096)
    assert c.payload_status(pay) == (0, -1) and pay.headers()[1][0].n_sat > 8
    # bad arguments
    with pytest.raises(api.AtomoError):
        c.set_entrywise_format(2, 0)
    with pytest.raises(api.AtomoError):
        c.set_entrywise_format(api.EW_COMPACT, -1)
    assert api.payload_bytes_entrywise_compact([100], 10, -1) == -1
    # a compact payload whose header was damaged is rejected by the decoder
    pay, _ = c.atomo_encode_entrywise([t], 4095.5, seed=5, k_cap=4096)
    hdr = pay.buf[:64].view(torch.int64)
    hdr[6] = 7                                            # unknown format
    assert not c.atomo_decode(pay)[0].any() and c.payload_status(pay)[0] == 8


def test_average_of_mixed_formats(pair, oracle):
    """The combine step reads each payload's own format: two explicit and two compact payloads."""
    import torch
    a, c = pair
    n, s, step = 10_000, 3000.0, 2
    gs = [np.random.default_rng([9, w]).standard_normal(n).astype(np.float32) for w in range(4)]
    gs[1][:50] *= 100.0                                   # some saturated atoms in a compact payload
    pays, singles = [], []
    for w, g in enumerate(gs):
        ctx = a if w % 2 == 0 else c
        pay, _ = ctx.atomo_encode_entrywise([torch.from_numpy(g).cuda()], s, seed=40 + w, step=step, k_cap=n)
        pays.append(pay)
        singles.append(ctx.atomo_decode(pay)[0].double())
    assert pays[1].headers()[1][0].n_sat > 0
    out = a.atomo_decode_average(pays)[0]
    # payload by payload in fp32, then one scaling: the same order in fp32 on the host
    acc = torch.zeros(n, dtype=torch.float32, device="cuda")
    for sgl in singles:
        acc += sgl.float()
    assert torch.equal(out, acc * 0.25)
    assert torch.equal(c.atomo_decode_average(pays[1:2])[0], singles[1].float())
