"""Seeded synthetic gradients shaped like the paper's CIFAR-scale CNN layers.

This module only *generates inputs*.  It contains none of the method's arithmetic
(no probabilities, no sampling, no decomposition of a gradient): both the CPU oracle
and the CUDA path receive the arrays produced here as plain fp32 buffers.

The paper trains ResNet-18 and VGG-11-BN on CIFAR-10 / SVHN (Table 2) and shows that a
convolution layer's gradient, seen as a matrix, has sharply decaying singular values
with a few dominant ones (Fig. 1).  Those datasets are not available here, so every
workload is a stand-in with the same layer shapes and a prescribed power-law spectrum
plus dense Gaussian noise:

    G = U diag(sigma) V^T + E,   U, V Haar-distributed with orthonormal columns.

All randomness comes from ``numpy.random.default_rng`` seeded from (workload, seed,
layer position); values are produced in float64 and rounded once to float32.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

__all__ = [
    "haar_columns", "lowrank_plus_noise", "LayerSpec", "RESNET18_LAYERS", "VGG11_LAYERS",
    "c1_spectral", "c1_entrywise", "c2_resnet18", "c3_vgg11", "c4_entrywise", "c5_stress",
    "c3_vgg11_layer", "c5_stress_layer",
    "layer_elements",
]


def _rng(tag: str, seed: int, index: int = 0) -> np.random.Generator:
    """Independent stream per (workload tag, user seed, layer position)."""
    return np.random.default_rng([zlib.crc32(tag.encode()), int(seed), int(index)])


def haar_columns(rng: np.random.Generator, rows: int, cols: int) -> np.ndarray:
    """``rows x cols`` matrix (cols <= rows) with orthonormal columns, Haar distributed.

    QR of a Gaussian matrix with the signs of diag(R) folded into Q.
    """
    assert cols <= rows
    q, r = np.linalg.qr(rng.standard_normal((rows, cols)))
    d = np.sign(np.diag(r))
    d[d == 0] = 1.0
    return q * d


def lowrank_plus_noise(rng: np.random.Generator, m: int, n: int, decay: float,
                       noise_rel: float | None = None, noise_std: float | None = None
                       ) -> np.ndarray:
    """fp32 ``m x n`` matrix with singular values ``i**-decay`` (before noise).

    ``noise_rel``: dense Gaussian noise scaled so that ||E||_F = noise_rel * ||G0||_F.
    ``noise_std``: dense Gaussian noise with that per-entry standard deviation.
    """
    r = min(m, n)
    sigma = np.arange(1, r + 1, dtype=np.float64) ** (-decay)
    u = haar_columns(rng, m, r)
    v = haar_columns(rng, n, r)
    g0 = (u * sigma) @ v.T
    if noise_rel is not None and noise_rel > 0:
        e = rng.standard_normal((m, n))
        e *= noise_rel * np.linalg.norm(g0) / np.linalg.norm(e)
        g0 = g0 + e
    elif noise_std is not None and noise_std > 0:
        g0 = g0 + noise_std * rng.standard_normal((m, n))
    return np.ascontiguousarray(g0.astype(np.float32))


@dataclass(frozen=True)
class LayerSpec:
    name: str
    rows: int   # c_out
    cols: int   # c_in * k * k


def _expand(spec: Sequence[Tuple[str, int, int, int]]) -> List[LayerSpec]:
    out: List[LayerSpec] = []
    for name, rows, cols, count in spec:
        for j in range(count):
            out.append(LayerSpec(f"{name}.{j}" if count > 1 else name, rows, cols))
    return out


# ResNet-18 (CIFAR variant) convolution gradients reshaped to c_out x (c_in*3*3), plus fc.
RESNET18_LAYERS: List[LayerSpec] = _expand([
    ("conv1", 64, 27, 1),
    ("layer1", 64, 576, 4),
    ("layer2.down", 128, 576, 1),
    ("layer2", 128, 1152, 3),
    ("layer3.down", 256, 1152, 1),
    ("layer3", 256, 2304, 3),
    ("layer4.down", 512, 2304, 1),
    ("layer4", 512, 4608, 3),
    ("fc", 10, 512, 1),
])

# VGG-11 convolutions (3x3, 64..512 channels) plus the three fully connected layers.
VGG11_LAYERS: List[LayerSpec] = _expand([
    ("conv1", 64, 27, 1),
    ("conv2", 128, 576, 1),
    ("conv3", 256, 1152, 1),
    ("conv4", 256, 2304, 1),
    ("conv5", 512, 2304, 1),
    ("conv6-8", 512, 4608, 3),
    ("fc6-7", 4096, 4096, 2),
    ("fc8", 10, 4096, 1),
])


def layer_elements(layers: Sequence[LayerSpec]) -> int:
    return int(sum(l.rows * l.cols for l in layers))


def c1_spectral(seed: int = 0) -> np.ndarray:
    """Config 1a: one 64x64 gradient, sigma_i = 1/i, noise N(0, 1e-4) (variance)."""
    return lowrank_plus_noise(_rng("c1a", seed), 64, 64, 1.0, noise_std=1e-2)


def c1_entrywise(seed: int = 0) -> np.ndarray:
    """Config 1b: 4096 i.i.d. N(0,1) entries."""
    return _rng("c1b", seed).standard_normal(4096).astype(np.float32)


def _layer_set(tag: str, layers: Sequence[LayerSpec], seed: int, decay: float,
               noise_rel: float) -> List[np.ndarray]:
    return [lowrank_plus_noise(_rng(tag, seed, i), l.rows, l.cols, decay, noise_rel=noise_rel)
            for i, l in enumerate(layers)]


def c2_resnet18(seed: int = 0, layers: Sequence[LayerSpec] = RESNET18_LAYERS) -> List[np.ndarray]:
    """Config 2: ResNet-18 layer set, sigma_i = i^-1.5, 1% (Frobenius) Gaussian noise."""
    return _layer_set("c2", layers, seed, 1.5, 0.01)


def c3_vgg11(seed: int = 0, layers: Sequence[LayerSpec] = VGG11_LAYERS) -> List[np.ndarray]:
    """Config 3: VGG-11 layer set, sigma_i = 1/i, 1% (Frobenius) Gaussian noise."""
    return _layer_set("c3", layers, seed, 1.0, 0.01)


def c3_vgg11_layer(seed: int, index: int) -> np.ndarray:
    """One layer of config 3 (the same matrix ``c3_vgg11(seed)[index]`` holds), without generating the others."""
    l = VGG11_LAYERS[index]
    return lowrank_plus_noise(_rng("c3", seed, index), l.rows, l.cols, 1.0, noise_rel=0.01)


def c5_stress_layer(seed: int, index: int, rows: int = 1024, cols: int = 4096) -> np.ndarray:
    """One matrix of config 5 (the same matrix ``c5_stress(seed)[index]`` holds)."""
    return lowrank_plus_noise(_rng("c5", seed, index), rows, cols, 1.0, noise_rel=0.005)


def c4_entrywise(seed: int = 0, n: int = 25_600_000) -> np.ndarray:
    """Config 4: flat gradient, i.i.d. Laplace(0, scale 1e-3)."""
    return _rng("c4", seed).laplace(0.0, 1e-3, size=n).astype(np.float32)


def paper_reshape(layer: Sequence[int]) -> tuple:
    """Section 6's own matricisation of a conv gradient of shape (x, y, k, k): x*y/2 rows by 2*k*k columns
    (a very tall matrix; an fc gradient stays as it is)."""
    if len(layer) == 2:
        return int(layer[0]), int(layer[1])
    x, y, k, _ = layer
    return (x * y) // 2, 2 * k * k


def c2_paper_reshape(seed: int = 0, convs: Optional[Sequence[Sequence[int]]] = None) -> List[np.ndarray]:
    """ResNet-18-shaped conv gradients in the paper's tall reshape (short side 2 k^2 = 18): sigma_i = i^-1.5,
    1 % noise, like config 2."""
    if convs is None:
        convs = [(64, 3, 3, 3), (64, 64, 3, 3), (128, 64, 3, 3), (256, 128, 3, 3)]
    out = []
    for i, c in enumerate(convs):
        m, n = paper_reshape(c)
        out.append(lowrank_plus_noise(_rng("c2r", seed, i), m, n, 1.5, noise_rel=0.01))
    return out


def torch_lowrank_plus_noise(m: int, n: int, decay: float, seed: int, device, noise_rel: float | None = None,
                             noise_std: float | None = None):
    """The recipe of ``lowrank_plus_noise`` generated on a CUDA device with torch's generator (fp64, rounded once
    to fp32): for benchmarks, where 96 Haar factors of order 4096 would take minutes on the host.  Not bit-equal
    to the numpy version (another generator); same distribution."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    r = min(m, n)

    def haar(rows, cols):
        q, rr = torch.linalg.qr(torch.randn(rows, cols, dtype=torch.float64, device=device, generator=gen))
        d = torch.sign(torch.diagonal(rr))
        d[d == 0] = 1.0
        return q * d

    sigma = torch.arange(1, r + 1, dtype=torch.float64, device=device) ** (-decay)
    g0 = (haar(m, r) * sigma) @ haar(n, r).T
    if noise_rel is not None and noise_rel > 0:
        e = torch.randn(m, n, dtype=torch.float64, device=device, generator=gen)
        g0 = g0 + e * (noise_rel * torch.linalg.norm(g0) / torch.linalg.norm(e))
    elif noise_std is not None and noise_std > 0:
        g0 = g0 + noise_std * torch.randn(m, n, dtype=torch.float64, device=device, generator=gen)
    return g0.to(torch.float32).contiguous()


def c5_stress(seed: int = 0, count: int = 96, rows: int = 1024, cols: int = 4096
              ) -> List[np.ndarray]:
    """Config 5: ``count`` matrices rows x cols, sigma_i = 1/i, 0.5% noise."""
    return [lowrank_plus_noise(_rng("c5", seed, i), rows, cols, 1.0, noise_rel=0.005)
            for i in range(count)]
