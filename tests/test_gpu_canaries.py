"""Guard words around every caller-owned buffer (payload, decoded outputs, the per-atom debug arrays): the kernels
may write inside the extents the header documents and nowhere else.  Stands in for a memory checker: the buffers
are carved out of larger allocations whose borders are filled with a pattern and compared after the calls."""
import ctypes

import numpy as np
import pytest

from paper_1806_04090_b200 import synth

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes on each side
PATTERN = 0xA5


@pytest.fixture(scope="module")
def atomo():
    import torch
    from paper_1806_04090_b200 import api
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    a = api.Atomo(0)
    yield a
    a.close()


class Guarded:
    """A byte buffer of `nbytes` (256-byte aligned start) between two guard regions."""

    def __init__(self, nbytes):
        import torch
        self.n = int(nbytes)
        self.raw = torch.full((GUARD + self.n + GUARD + 256,), PATTERN, dtype=torch.uint8, device="cuda")
        off = (-self.raw.data_ptr() - GUARD) % 256
        self.lo = off
        self.view = self.raw[off + GUARD: off + GUARD + self.n]

    def typed(self, dtype, shape):
        return self.view.view(dtype).view(shape)

    def intact(self):
        before = self.raw[: self.lo + GUARD]
        after = self.raw[self.lo + GUARD + self.n:]
        return bool((before == PATTERN).all()) and bool((after == PATTERN).all())


def _spectral(atomo, mats, s, k_cap):
    import torch
    from paper_1806_04090_b200 import api
    shapes = [m.shape for m in mats]
    ts = [torch.from_numpy(m).cuda() for m in mats]
    pay_g = Guarded(api.payload_bytes_spectral(shapes, k_cap))
    pay, dbg = atomo.atomo_encode_spectral(ts, s, seed=3, step=1, k_cap=k_cap, payload=pay_g.view)
    outs_g = [Guarded(4 * m.size) for m in mats]
    outs = [g.typed(torch.float32, m.shape) for g, m in zip(outs_g, mats)]
    atomo.atomo_decode(pay, out=outs)
    torch.cuda.synchronize()
    assert atomo.payload_status(pay)[0] == 0
    assert pay_g.intact(), "encode or decode wrote outside the payload"
    for g in outs_g:
        assert g.intact(), "decode wrote outside an output"
    assert all(torch.isfinite(o).all() for o in outs)


def test_spectral_small_layers(atomo):
    L = synth.RESNET18_LAYERS
    _spectral(atomo, synth.c2_resnet18(0, [L[0], L[1], L[9], L[17]]), 2.0, k_cap=16)


def test_spectral_large_and_ragged_layers(atomo):
    rng = np.random.default_rng(5)
    mats = [synth.lowrank_plus_noise(rng, 601, 1203, 1.0, noise_rel=0.01), synth.lowrank_plus_noise(rng, 1030, 777, 1.0, noise_rel=0.01),
            synth.lowrank_plus_noise(rng, 33, 100, 1.0, noise_rel=0.01)]
    for ctas in (0, 1):
        try:
            atomo.set_tridiag_ctas(ctas)
            _spectral(atomo, mats, 3.0, k_cap=24)
        finally:
            atomo.set_tridiag_ctas(0)


@pytest.mark.parametrize("compact", [False, True])
def test_entrywise(atomo, compact):
    import torch
    from paper_1806_04090_b200 import api
    n = 1_000_003
    g = torch.from_numpy(synth.c4_entrywise(1, n)).cuda()
    s = 0.01 * n
    kc = int(1.1 * s) + 100
    try:
        if compact:
            atomo.set_entrywise_format(api.EW_COMPACT, 64)
            nbytes = api.payload_bytes_entrywise_compact([n], kc, 64)
        else:
            nbytes = api.payload_bytes_entrywise([n], kc)
        pay_g = Guarded(nbytes)
        pay, _ = atomo.atomo_encode_entrywise([g], s, seed=9, step=2, k_cap=kc, payload=pay_g.view)
        out_g = Guarded(4 * n)
        out = out_g.typed(torch.float32, (n,))
        atomo.atomo_decode(pay, out=[out])
        torch.cuda.synchronize()
    finally:
        atomo.set_entrywise_format(api.EW_EXPLICIT, 0)
    assert atomo.payload_status(pay)[0] == 0
    assert pay_g.intact() and out_g.intact()
    assert int((out != 0).sum()) == pay.headers()[1][0].k
