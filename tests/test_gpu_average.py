"""GPU: atomo_decode_average (the combine step of data-parallel training, Section 2 of the paper) through the
C ABI, against the mean of single-payload decodes and against the fp64 oracle."""
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


def _spectral_layers():
    shapes = [(64, 27), (64, 576), (10, 512), (300, 40), (128, 1152)]
    return [synth.lowrank_plus_noise(np.random.default_rng([5, i]), m, n, 1.5, noise_rel=0.01) for i, (m, n) in enumerate(shapes)]


def test_spectral_average_matches_mean_of_decodes(atomo):
    import torch
    from paper_1806_04090_b200 import api
    mats = _spectral_layers()
    ts = [torch.from_numpy(m).cuda() for m in mats]
    pays, singles = [], []
    for worker in range(3):                               # three workers: same gradients here, different seeds
        buf = torch.empty(api.payload_bytes_spectral([m.shape for m in mats], 16), dtype=torch.uint8, device="cuda")
        pay, _ = atomo.atomo_encode_spectral(ts, 3.0, seed=100 + worker, step=7, k_cap=16, payload=buf)
        assert max(h.status for h in pay.headers()[1]) == 0
        pays.append(pay)
        singles.append([o.clone() for o in atomo.atomo_decode(pay)])
    avg = atomo.atomo_decode_average(pays)
    for l in range(len(mats)):
        want = (singles[0][l].double() + singles[1][l].double() + singles[2][l].double()) / 3.0
        scale = float(want.abs().max())
        assert float((avg[l].double() - want).abs().max()) <= 2e-6 * scale + 1e-12
    # one payload: the plain decode, bit for bit
    one = atomo.atomo_decode_average(pays[:1])
    for l in range(len(mats)):
        assert torch.equal(one[l], singles[0][l])


def test_spectral_average_against_oracle(atomo, oracle):
    """The averaging decode against the oracle's definition of the combine step: the mean over the workers of the
    oracle's decode (Eq. 2) of each worker's own kept atoms."""
    import torch
    from paper_1806_04090_b200 import api
    mats = _spectral_layers()
    ts = [torch.from_numpy(m).cuda() for m in mats]
    pays = []
    for worker in range(4):
        buf = torch.empty(api.payload_bytes_spectral([m.shape for m in mats], 16), dtype=torch.uint8, device="cuda")
        pay, _ = atomo.atomo_encode_spectral(ts, 2.5, seed=300 + worker, step=2, k_cap=16, payload=buf)
        assert max(h.status for h in pay.headers()[1]) == 0
        pays.append(pay)
    avg = atomo.atomo_decode_average(pays)
    for l, G in enumerate(mats):
        want = np.zeros(G.shape)
        for pay in pays:
            arr = pay.layer_arrays(l)
            want += oracle.decode_spectral(arr["coef"], arr["U"], arr["V"])
        want /= len(pays)
        assert parity.rel(avg[l].cpu().numpy(), want) <= 1e-5


def test_entrywise_average_against_oracle(atomo, oracle):
    import torch
    from paper_1806_04090_b200 import api
    n, s, step = 10_000, 3000.0, 2                        # ragged tail tile; 30 % kept, so the payloads' indices collide
    workers = 4
    gs = [np.random.default_rng([9, w]).standard_normal(n).astype(np.float32) for w in range(workers)]
    pays, ref = [], np.zeros(n, dtype=np.float64)
    carved = 0
    for w, g in enumerate(gs):
        buf = torch.empty(api.payload_bytes_entrywise([n], n), dtype=torch.uint8, device="cuda")
        pay, _ = atomo.atomo_encode_entrywise([torch.from_numpy(g).cuda()], s, seed=40 + w, step=step, k_cap=n, payload=buf)
        pays.append(pay)
        enc = oracle.encode_entrywise(g, s, seed=40 + w, step=step)
        arr = pay.layer_arrays(0)
        if not np.array_equal(arr["idx"].astype(np.int64), enc["idx"]):
            # a draw within the carve-out of p_i decided differently in fp32: use the payload's own kept set
            carved += 1
            dense = np.zeros(n); dense[arr["idx"].astype(np.int64)] = arr["val"]
            ref += dense
        else:
            ref += oracle.decode_entrywise(n, enc["idx"], enc["val"])
    ref /= workers
    out = atomo.atomo_decode_average(pays)[0].cpu().numpy()
    print(f"workers whose kept set differed from the oracle's inside the carve-out: {carved}")
    assert parity.rel(out, ref) <= 1e-6
    # exact structure: an element is non-zero iff some payload kept it
    kept_any = np.zeros(n, dtype=bool)
    for pay in pays:
        kept_any[pay.layer_arrays(0)["idx"].astype(np.int64)] = True
    assert not out[~kept_any].any()
    single = atomo.atomo_decode(pays[0])[0]
    assert torch.equal(atomo.atomo_decode_average(pays[:1])[0], single)


def test_average_argument_and_payload_errors(atomo):
    import ctypes
    import torch
    from paper_1806_04090_b200 import api
    g = torch.from_numpy(synth.c1_entrywise(0)).cuda()
    pay_e, _ = atomo.atomo_encode_entrywise([g], 64.0, seed=1, k_cap=g.numel())
    G = torch.from_numpy(synth.c1_spectral(0)).cuda()
    pay_s, _ = atomo.atomo_encode_spectral([G], 2.0, seed=1, k_cap=16)
    with pytest.raises(ValueError):
        atomo.atomo_decode_average([])
    with pytest.raises(ValueError):
        atomo.atomo_decode_average([pay_e, pay_s])
    # C level: no payloads -> invalid argument; an entry-wise payload offered as spectral -> zeros and a status word
    rows = (ctypes.c_int64 * 1)(64); cols = (ctypes.c_int64 * 1)(64)
    out = torch.full((64, 64), 7.0, dtype=torch.float32, device="cuda")
    ptrs = (ctypes.c_void_p * 1)(out.data_ptr())
    pays = (ctypes.c_void_p * 1)(pay_e.buf.data_ptr())
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert atomo.lib.atomo_decode_average(atomo._h, api.KIND_SPECTRAL, pays, 0, rows, cols, ptrs, 1, stream) == 1   # ATOMO_ERR_INVALID_ARG
    assert atomo.lib.atomo_decode_average(atomo._h, api.KIND_SPECTRAL, pays, 1, rows, cols, ptrs, 1, stream) == 0
    torch.cuda.synchronize()
    assert not out.any()
    assert pay_e.headers()[1][0].status == 8   # ATOMO_ERR_PAYLOAD
