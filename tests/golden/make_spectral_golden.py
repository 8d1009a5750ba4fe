"""Writes the stored oracle results for the large spectral layers (configs 3 and 5).

The fp64 one-sided Jacobi SVD of the oracle takes minutes for a 1024 x 4096 matrix and hours for a
4096 x 4096 one, so its results for a few seeded layers are computed once, here, and stored beside
this script; the GPU parity tests load them.  This script calls only ``oracle/`` and the seeded
input generators (``synth``), never the CUDA library.

    python tests/golden/make_spectral_golden.py c5 0        # config 5, matrix 0  -> spectral_c5_m0.npz
    python tests/golden/make_spectral_golden.py c5 1
    python tests/golden/make_spectral_golden.py c3 8        # config 3, layer 8 (4096 x 4096)
    python tests/golden/make_spectral_golden.py c5small 0   # 256 x 1024 stand-in, seconds (self-test of the format)

Stored per case: shape, generator seed, CRC-32 of the fp32 input bytes, the Philox seed / step /
layer position the draws were made with, sigma (all r values, fp64), and per budget s (Eq. 2,
Algorithm 1): p (fp64), the mask, kept ranks, coef = sigma_i / p_i and the kept singular vectors
U_S (short or long side as the matrix lies), V_S, all fp64, plus the number of sweeps the SVD took.
"""
from __future__ import annotations

import os
import sys
import time
import zlib

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import atomo_oracle as oracle                      # noqa: E402
from paper_1806_04090_b200 import synth                        # noqa: E402  (input generators only)

# case name -> (generator, generator seed, budgets, Philox seed, step)
CASES = {
    "c5": dict(gen=lambda seed, i: synth.c5_stress_layer(seed, i), gen_seed=0, budgets=(2.0, 4.0, 8.0),
               philox_seed=0x5EED0005, step=3),
    "c3": dict(gen=lambda seed, i: synth.c3_vgg11_layer(seed, i), gen_seed=0, budgets=(1.0, 2.0, 3.0),
               philox_seed=0x5EED0003, step=7),
    "c5small": dict(gen=lambda seed, i: synth.c5_stress_layer(seed, i, rows=256, cols=1024), gen_seed=0,
                    budgets=(2.0, 4.0, 8.0), philox_seed=0x5EED0005, step=3),
}


def path_of(case: str, index: int) -> str:
    return os.path.join(HERE, f"spectral_{case}_m{index}.npz")


def main(case: str, index: int) -> None:
    cfg = CASES[case]
    G = cfg["gen"](cfg["gen_seed"], index)
    t0 = time.time()
    U, sigma, V = oracle.jacobi_svd(G)
    took = time.time() - t0
    out = dict(shape=np.array(G.shape, dtype=np.int64), gen_seed=np.int64(cfg["gen_seed"]),
               index=np.int64(index), crc32=np.uint32(zlib.crc32(G.tobytes())),
               philox_seed=np.uint64(cfg["philox_seed"]), step=np.int64(cfg["step"]), layer=np.int64(index),
               budgets=np.array(cfg["budgets"]), sigma=sigma, svd_seconds=np.float64(took))
    for s in cfg["budgets"]:
        enc = oracle.encode_spectral_from_svd(U, sigma, V, s, cfg["philox_seed"], step=cfg["step"], layer=index)
        tag = f"s{s:g}"
        out[f"{tag}_p"] = enc["p"]
        out[f"{tag}_mask"] = np.packbits(enc["mask"])
        out[f"{tag}_idx"] = enc["idx"]
        out[f"{tag}_coef"] = enc["coef"]
        out[f"{tag}_U_S"] = enc["U_S"]
        out[f"{tag}_V_S"] = enc["V_S"]
        out[f"{tag}_n_s"] = np.int64(enc["n_s"])
    np.savez_compressed(path_of(case, index), **out)
    print(f"{case} m{index}: {G.shape}, SVD {took:.1f} s, kept {[int(out[f's{s:g}_idx'].size) for s in cfg['budgets']]}")


if __name__ == "__main__":
    main(sys.argv[1], int(sys.argv[2]))
