"""The allocation-free spectral decode (atomo_decode_spectral_static) against atomo_decode.

Some processes cannot call cudaMalloc where they decode: the framework's caching allocator may
already hold the whole GPU, and cudaMalloc synchronises the device.  That entry point keeps its
per-call tables in a fixed array inside the library instead of the context's workspace.  It runs
the same decode kernel, so its output must equal atomo_decode's bit for bit -- on two calls in a
row with different batches, because the shared array still holds the first call's tables when
the second one starts.  The file name sorts last so that a run stopping at the first failure has
already run every other test.
"""
import numpy as np
import pytest

from paper_1806_04090_b200 import synth

pytestmark = pytest.mark.gpu


def test_static_decode_matches_decode_twice_in_a_row():
    import torch
    from paper_1806_04090_b200 import api
    assert torch.cuda.is_available()
    a = api.Atomo(0)
    L = synth.RESNET18_LAYERS
    batches = [synth.c2_resnet18(0, [L[1], L[5], L[9], L[17]]),            # wide layers, 4 of them
               [synth.c1_spectral(0), synth.c2_resnet18(1, [L[0]])[0]]]     # square and tall, 2 layers
    for call, mats in enumerate(batches):
        ts = [torch.from_numpy(G).cuda() for G in mats]
        pay, _ = a.atomo_encode_spectral(ts, 3.0, seed=40 + call, step=call, k_cap=32)
        assert a.payload_status(pay)[0] == 0
        assert sum(h.k for h in pay.headers()[1]) > 0
        want = a.atomo_decode(pay)
        got = [torch.full_like(w, float("nan")) for w in want]               # every element must be written
        api.atomo_decode_spectral_static(pay, got)
        torch.cuda.synchronize()
        for w, g in zip(want, got):
            assert torch.equal(w, g)
    a.close()


def test_static_decode_rejects_oversized_batches():
    import torch
    from paper_1806_04090_b200 import api
    a = api.Atomo(0)
    G = torch.from_numpy(synth.c1_spectral(0)).cuda()
    pay, _ = a.atomo_encode_spectral([G], 2.0, seed=1, k_cap=8)
    # more layers than the fixed table holds (every output is a real 64 x 64 buffer: nothing depends on the refusal)
    big = api.Payload(pay.buf, api.KIND_SPECTRAL, [(64, 64)] * 65, 8, a)
    with pytest.raises(api.AtomoError) as e:
        api.atomo_decode_spectral_static(big, [torch.empty(64, 64, device="cuda") for _ in range(65)])
    assert e.value.code == 3
    # more output tiles than the fixed table holds: 8193 row tiles of 64 x 1024, in a buffer of the full size (2 MB)
    huge = api.Payload(pay.buf, api.KIND_SPECTRAL, [(64 * 8193, 1)], 8, a)
    with pytest.raises(api.AtomoError) as e:
        api.atomo_decode_spectral_static(huge, [torch.empty(64 * 8193, 1, device="cuda")])
    assert e.value.code == 3
    # the binding refuses outputs that are too short, strided, of another type or on the host before the C call
    ok = api.Payload(pay.buf, api.KIND_SPECTRAL, [(64, 64)], 8, a)
    for bad in (torch.empty(1, device="cuda"), torch.empty(64, 128, device="cuda")[:, ::2],
                torch.empty(64, 64, device="cuda", dtype=torch.float64), torch.empty(64, 64)):
        with pytest.raises(ValueError):
            api.atomo_decode_spectral_static(ok, [bad])
    a.close()
