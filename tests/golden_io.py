"""Loader for the stored oracle results of the large spectral layers (written by
``tests/golden/make_spectral_golden.py``, which calls only the oracle and the seeded input generators)."""
from __future__ import annotations

import os
import zlib

import numpy as np

from paper_1806_04090_b200 import synth

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")

_GEN = {
    "c5": lambda seed, i: synth.c5_stress_layer(seed, i),
    "c3": lambda seed, i: synth.c3_vgg11_layer(seed, i),
    "c5small": lambda seed, i: synth.c5_stress_layer(seed, i, rows=256, cols=1024),
}


def have(case: str, index: int) -> bool:
    return os.path.exists(os.path.join(GOLDEN, f"spectral_{case}_m{index}.npz"))


def load(case: str, index: int):
    """Returns (G fp32, meta dict, {s: enc dict in the oracle's encode_spectral layout without the words})."""
    z = np.load(os.path.join(GOLDEN, f"spectral_{case}_m{index}.npz"))
    G = _GEN[case](int(z["gen_seed"]), int(z["index"]))
    assert tuple(z["shape"]) == G.shape
    assert int(z["crc32"]) == zlib.crc32(G.tobytes()), "the input generator no longer reproduces the stored case"
    r = min(G.shape)
    meta = dict(philox_seed=int(z["philox_seed"]), step=int(z["step"]), layer=int(z["layer"]),
                budgets=[float(s) for s in z["budgets"]], svd_seconds=float(z["svd_seconds"]))
    encs = {}
    for s in meta["budgets"]:
        t = f"s{s:g}"
        encs[s] = dict(sigma=z["sigma"], p=z[f"{t}_p"], mask=np.unpackbits(z[f"{t}_mask"])[:r].astype(bool),
                       idx=z[f"{t}_idx"], coef=z[f"{t}_coef"], U_S=z[f"{t}_U_S"], V_S=z[f"{t}_V_S"],
                       n_s=int(z[f"{t}_n_s"]))
    return G, meta, encs
