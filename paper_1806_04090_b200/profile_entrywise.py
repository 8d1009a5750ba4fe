"""Small driver for profiling the entry-wise path on config 4 (25.6M Laplace elements): a few encode + decode
steps at s = 1 % of the length.  Run it under ncu to capture ew_solve / ew_sample_pack / ew_decode."""
from __future__ import annotations

import sys

import torch

from . import api, synth


def main(steps: int = 4) -> None:
    a = api.Atomo(0)
    g = torch.from_numpy(synth.c4_entrywise(0)).cuda()
    n = g.numel()
    s = 0.01 * n
    k_cap = int(s * 1.05) + 1000
    payload = torch.empty(api.payload_bytes_entrywise([n], k_cap), dtype=torch.uint8, device="cuda")
    out = torch.empty_like(g)
    for i in range(steps):
        pay, _ = a.atomo_encode_entrywise([g], s, seed=7, step=i, k_cap=k_cap, payload=payload)
        a.atomo_decode(pay, out=[out])
    torch.cuda.synchronize()
    print("status", max(h.status for h in pay.headers()[1]), "k", pay.headers()[1][0].k)
    a.close()


if __name__ == "__main__":
    main(int(sys.argv[1]) if len(sys.argv) > 1 else 4)
