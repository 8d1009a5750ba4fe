"""TEST INFRASTRUCTURE -- the CPU oracle for the ATOMO encode/decode path (fp64).

A plain, slow, double-precision statement of what the CUDA library must compute, written
from the paper.  Only ``tests/``, the smoke check and the CPU-baseline leg of ``bench.py``
may import it; the product never does, and this file imports nothing from the product.

What each function follows:

* ``atomo_probabilities``  -- the solution of Eq. (3) in the closed form of Appendix B (what Algorithm 1 computes),
  with the readings below.
* ``bernoulli_words`` / ``sample_mask`` -- the independent Bernoulli(p_i) draws of Eq. (2).
  The paper fixes only the distribution; generator, key and counter layout are this
  project's definition (Philox4x32-10, Salmon et al., SC'11).  Parity of the *stream*
  is therefore pinned by that publication's known-answer vectors, not by the paper.
* ``lq_budget`` -- Section 4's budget s = ||g||_1 / ||g||_q (QSGD for q = 2, TernGrad for q = inf).
* ``jacobi_svd`` -- the SVD  X = sum sigma_i u_i v_i^T  of Section 5 (one-sided Jacobi, C).
* ``encode_entrywise`` / ``encode_spectral`` -- Eq. (2): keep atom i iff t_i = 1, with
  weight lambda_i / p_i.
* ``decode_entrywise`` / ``decode_spectral`` -- Eq. (2) summed back to a dense gradient.

Readings of the paper where it is silent, garbled or inconsistent:

* Algorithm 1 prints  sum_{j=i}^n |lambda_i| ; the summand is |lambda_j|
  (Definition 1 and the closed form of Appendix B agree on that).
* lambda_i = 0  gives  p_i = 0  (Appendix B, item 2): such an atom is never drawn, so
  sum(p) = min(s, number of non-zero atoms).
* Any s > 0 is accepted; s >= n gives p = 1 on every non-zero atom (Appendix B, item 1).
* Ties among equal |lambda| cannot change p (p depends on |lambda_i| only); the sort is stable.
* Budget s is a real number (the QSGD / TernGrad budgets of Section 4 are not integers).

Pins (see tests/test_oracle_*.py): closed forms of Lemma 2 / Appendix B, the invariants
sum(p)=s and 0<=p<=1, brute-force minimisation of Eq. (3) on <= 6 atoms, the QSGD and
TernGrad special cases of Section 4, Lemma 1's moments by Monte Carlo, Table 1's second
moments, Appendix C's tight examples for the SVD, a library SVD as a third opinion, and
the published Philox4x32-10 known-answer vectors.  No function here is "parity unpinned"
except the counter layout of ``bernoulli_words`` (a project definition the paper has no
counterpart for; the generator itself is pinned).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libatomo_oracle.so")
_lib = None

KIND_SPECTRAL = 0
KIND_ENTRYWISE = 1


def build(force: bool = False) -> str:
    """Compile the C part of the oracle (gcc -O2, no BLAS)."""
    src = os.path.join(_HERE, "jacobi_svd.c")
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-o", _LIB_PATH, src, "-lm"])
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB_PATH)
        lib.oracle_jacobi_svd.restype = ctypes.c_int
        lib.oracle_jacobi_svd.argtypes = [
            ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_double, ctypes.c_int]
        _lib = lib
    return _lib


# --------------------------------------------------------------------------------------
# Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3")
# --------------------------------------------------------------------------------------
_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0: int, k1: int):
    """Ten rounds of Philox-4x32 on arrays of counter words; returns four uint32 arrays."""
    c0 = np.asarray(c0, dtype=np.uint64) & _MASK32
    c1 = np.asarray(c1, dtype=np.uint64) & _MASK32
    c2 = np.asarray(c2, dtype=np.uint64) & _MASK32
    c3 = np.asarray(c3, dtype=np.uint64) & _MASK32
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _W0) & 0xFFFFFFFF
            k1 = (k1 + _W1) & 0xFFFFFFFF
        prod0 = _M0 * c0            # 32x32 -> 64 bit, exact in uint64
        prod1 = _M1 * c2
        hi0, lo0 = prod0 >> np.uint64(32), prod0 & _MASK32
        hi1, lo1 = prod1 >> np.uint64(32), prod1 & _MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)), lo1, (hi0 ^ c3 ^ np.uint64(k1)), lo0
    return (c0.astype(np.uint32), c1.astype(np.uint32), c2.astype(np.uint32), c3.astype(np.uint32))


def bernoulli_words(seed: int, step: int, layer: int, kind: int, n_atoms: int) -> np.ndarray:
    """The 32-bit uniform word x_i that decides atom i.

    Project definition (the paper has no counterpart): key = (seed low 32, seed high 32);
    counter = (block low 32, block high 32, layer, (kind << 31) | (step & 0x7fffffff)) with
    block = i >> 2; atom i takes output word i & 3 of its block.  ``layer`` is the position of
    the layer (or vector) inside one encode call; spectral atoms are indexed by rank in
    descending sigma, entry-wise atoms by flat element index.
    """
    n_blocks = (int(n_atoms) + 3) // 4
    blk = np.arange(n_blocks, dtype=np.uint64)
    w = philox4x32_10(blk & _MASK32, blk >> np.uint64(32),
                      np.full(n_blocks, int(layer) & 0xFFFFFFFF, dtype=np.uint64),
                      np.full(n_blocks, ((int(kind) & 1) << 31) | (int(step) & 0x7FFFFFFF), dtype=np.uint64),
                      int(seed) & 0xFFFFFFFF, (int(seed) >> 32) & 0xFFFFFFFF)
    return np.stack(w, axis=1).reshape(-1)[: int(n_atoms)]


def bernoulli_threshold(p: np.ndarray) -> np.ndarray:
    """floor(p * 2^32) as uint64 (exact for double p in [0, 1])."""
    return np.floor(np.asarray(p, dtype=np.float64) * 4294967296.0).astype(np.uint64)


def sample_mask(p: np.ndarray, words: np.ndarray) -> np.ndarray:
    """t_i ~ Bernoulli(p_i) of Eq. (2), decided in integers: t_i = 1 if p_i >= 1, else
    [x_i < floor(p_i 2^32)].  p_i = 0 is never drawn."""
    p = np.asarray(p, dtype=np.float64)
    return (p >= 1.0) | (words.astype(np.uint64) < bernoulli_threshold(p))


# --------------------------------------------------------------------------------------
# Algorithm 1
# --------------------------------------------------------------------------------------
def atomo_probabilities(lam: np.ndarray, s: float) -> Tuple[np.ndarray, int, float]:
    """The p solving  min sum lambda_i^2 / p_i,  0 < p_i <= 1,  sum p_i = s  (Eq. 3), from the closed form of
    Appendix B: with |lambda_1| >= ... >= |lambda_n| and tail_i = sum_{j >= i} |lambda_j|, n_s is the first count of
    leading atoms for which the rest is (s - n_s)-balanced, |lambda_{n_s+1}| (s - n_s) <= tail_{n_s+1}; those n_s atoms
    get p = 1 and the rest p_i = |lambda_i| (s - n_s) / tail_{n_s+1}.  (Algorithm 1 reaches the same n_s one atom at a
    time.)

    Returns (p in the caller's order, n_s, c = tail_{n_s+1} / (s - n_s), the common weight |lambda_i| / p_i of the atoms
    with p < 1; c = 0 when that tail is empty or all zero).
    """
    if not (s > 0.0) or not np.isfinite(s):
        raise ValueError("sparsity budget s must be a positive finite number")
    a = np.abs(np.asarray(lam, dtype=np.float64)).reshape(-1)
    n = a.size
    order = np.argsort(-a, kind="stable")          # |lambda_1| >= ... >= |lambda_n|
    a_sorted = a[order]
    tail = np.cumsum(a_sorted[::-1])[::-1] if n else a_sorted      # tail[i] = sum_{j >= i} |lambda_j|, from the small end
    budget = float(s) - np.arange(n, dtype=np.float64)             # what is left after i atoms were given p = 1
    balanced = a_sorted * budget <= tail                           # the remaining atoms are budget-balanced from i on
    # an atom with lambda = 0 is never given p = 1: where it comes first its tail is 0 and the test holds (0 <= 0), so a
    # budget s >= n ends with p = 1 exactly on the non-zero atoms
    n_s = int(np.argmax(balanced)) if balanced.any() else n
    p_sorted = np.zeros(n, dtype=np.float64)
    p_sorted[:n_s] = 1.0
    c = 0.0
    if n_s < n and tail[n_s] > 0.0:
        p_sorted[n_s:] = a_sorted[n_s:] * budget[n_s] / tail[n_s]
        c = float(tail[n_s] / budget[n_s])
    p = np.empty(n, dtype=np.float64)
    p[order] = p_sorted
    return p, n_s, float(c)


# --------------------------------------------------------------------------------------
# SVD
# --------------------------------------------------------------------------------------
def lq_budget(g: np.ndarray, q: float) -> float:
    """Section 4: the budget s = ||g||_1 / ||g||_q at which entry-wise ATOMO is the l_q quantiser
    (q = 2: QSGD, q = inf: TernGrad).  Plain definition in fp64; a zero vector gives 0."""
    a = np.abs(np.asarray(g, dtype=np.float64).reshape(-1))
    if not (q >= 1.0):
        raise ValueError("q must be >= 1")
    l1 = float(a.sum())
    if l1 == 0.0:
        return 0.0
    nq = float(a.max()) if np.isinf(q) else float((a ** q).sum() ** (1.0 / q))
    return l1 / nq


def jacobi_svd(G: np.ndarray, tol: float = 1e-15, max_sweeps: int = 60):
    """Thin SVD of G (m x n) -> (U m x r, sigma r descending, V n x r), r = min(m, n)."""
    G = np.ascontiguousarray(np.asarray(G, dtype=np.float64))
    m, n = G.shape
    r = min(m, n)
    U = np.zeros((m, r)); sig = np.zeros(r); V = np.zeros((n, r))
    rc = _load().oracle_jacobi_svd(G.ctypes.data, m, n, U.ctypes.data, sig.ctypes.data,
                                   V.ctypes.data, float(tol), int(max_sweeps))
    if rc < 0:
        raise RuntimeError(f"one-sided Jacobi did not converge (code {rc})")
    return U, sig, V


# --------------------------------------------------------------------------------------
# encode / decode
# --------------------------------------------------------------------------------------
def encode_entrywise(g: np.ndarray, s: float, seed: int, step: int = 0, layer: int = 0) -> Dict:
    """Entry-wise ATOMO: atoms e_i with lambda_i = g_i.  Kept entries in ascending index."""
    g64 = np.asarray(g, dtype=np.float64).reshape(-1)
    p, n_s, c = atomo_probabilities(g64, s)
    words = bernoulli_words(seed, step, layer, KIND_ENTRYWISE, g64.size)
    mask = sample_mask(p, words)
    idx = np.flatnonzero(mask)
    val = g64[idx] / p[idx]
    return dict(p=p, n_s=n_s, c=c, words=words, mask=mask, idx=idx.astype(np.int64), val=val)


def decode_entrywise(n: int, idx: np.ndarray, val: np.ndarray) -> np.ndarray:
    out = np.zeros(int(n), dtype=np.float64)
    out[np.asarray(idx, dtype=np.int64)] = val
    return out


def encode_spectral_from_svd(U, sigma, V, s: float, seed: int, step: int = 0, layer: int = 0) -> Dict:
    """Spectral ATOMO downstream of a given SVD: atoms u_i v_i^T with lambda_i = sigma_i."""
    sigma = np.asarray(sigma, dtype=np.float64)
    p, n_s, c = atomo_probabilities(sigma, s)
    words = bernoulli_words(seed, step, layer, KIND_SPECTRAL, sigma.size)
    mask = sample_mask(p, words)
    idx = np.flatnonzero(mask)
    coef = sigma[idx] / p[idx]
    return dict(sigma=sigma, p=p, n_s=n_s, c=c, words=words, mask=mask, idx=idx.astype(np.int64),
                coef=coef, U_S=np.asarray(U)[:, idx].copy(), V_S=np.asarray(V)[:, idx].copy())


def encode_spectral(G: np.ndarray, s: float, seed: int, step: int = 0, layer: int = 0) -> Dict:
    U, sigma, V = jacobi_svd(G)
    out = encode_spectral_from_svd(U, sigma, V, s, seed, step, layer)
    out.update(U=U, V=V)
    return out


def decode_spectral(coef: np.ndarray, U_S: np.ndarray, V_S: np.ndarray) -> np.ndarray:
    """sum_k coef_k u_k v_k^T  (zero matrix if nothing was kept)."""
    U_S = np.asarray(U_S, dtype=np.float64)
    V_S = np.asarray(V_S, dtype=np.float64)
    return (U_S * np.asarray(coef, dtype=np.float64)) @ V_S.T
