"""Seeded value generators and the five benchmark/test configurations.

Every generator returns float32.  The draws use float32 numpy fast paths so
that a 143.7 M-element bucket takes seconds rather than minutes to build.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence

import numpy as np

from .shapes import numel, resnet50_shapes, vgg19_shapes


@dataclass
class Bucket:
    """A flat fp32 bucket of T tensors: tensor t is values[offsets[t]:offsets[t+1]]."""

    values: np.ndarray  # float32, shape (N,)
    offsets: np.ndarray  # int64, shape (T+1,), offsets[0] == 0
    names: List[str]

    @property
    def num_tensors(self) -> int:
        return len(self.offsets) - 1

    @property
    def total(self) -> int:
        return int(self.offsets[-1])

    def tensor(self, t: int) -> np.ndarray:
        return self.values[int(self.offsets[t]) : int(self.offsets[t + 1])]


def offsets_from_sizes(sizes: Sequence[int]) -> np.ndarray:
    off = np.zeros(len(sizes) + 1, dtype=np.int64)
    np.cumsum(np.asarray(sizes, dtype=np.int64), out=off[1:])
    return off


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def gaussian(rng: np.random.Generator, n: int, sigma: float) -> np.ndarray:
    return rng.standard_normal(n, dtype=np.float32) * np.float32(sigma)


def laplace(rng: np.random.Generator, n: int, b: float) -> np.ndarray:
    mag = rng.standard_exponential(n, dtype=np.float32)
    neg = rng.random(n, dtype=np.float32) < np.float32(0.5)
    mag *= np.float32(b)
    np.negative(mag, where=neg, out=mag)
    return mag


def student_t(rng: np.random.Generator, n: int, nu: float, scale: float) -> np.ndarray:
    z = rng.standard_normal(n, dtype=np.float32)
    g = rng.standard_gamma(nu / 2.0, n, dtype=np.float32)  # chi2_nu = 2 g
    np.maximum(g, np.float32(1e-30), out=g)
    z *= np.sqrt(np.float32(nu) / (np.float32(2.0) * g))
    z *= np.float32(scale)
    return z


def mixture(rng: np.random.Generator, n: int, w: float, sigma_a: float, sigma_b: float) -> np.ndarray:
    """w * N(0, sigma_a) + (1 - w) * N(0, sigma_b), component chosen per element."""
    pick_a = rng.random(n, dtype=np.float32) < np.float32(w)
    z = rng.standard_normal(n, dtype=np.float32)
    return z * np.where(pick_a, np.float32(sigma_a), np.float32(sigma_b)).astype(np.float32)


def config1(seed: int = 0) -> Bucket:
    """One tensor of 65,536 i.i.d. Laplace(0, b=1e-3) values."""
    v = laplace(_rng(seed), 65536, 1e-3)
    return Bucket(v, offsets_from_sizes([v.size]), ["laplace"])


def config2(seed: int = 2) -> Bucket:
    """Four tensors: 1M Gaussian, 256K Laplace, 64K Student-t(3), 4K 90/10 Gaussian mixture."""
    rng = _rng(seed)
    parts = [
        gaussian(rng, 1 << 20, 1e-3),
        laplace(rng, 1 << 18, 1e-3),
        student_t(rng, 1 << 16, 3.0, 1e-3),
        mixture(rng, 1 << 12, 0.9, 1e-4, 1e-2),
    ]
    return Bucket(
        np.concatenate(parts),
        offsets_from_sizes([p.size for p in parts]),
        ["gaussian", "laplace", "student_t3", "mixture"],
    )


def _log_uniform_scales(n: int, seed: int) -> np.ndarray:
    return 10.0 ** _rng(seed).uniform(-5.0, -2.0, size=n)


def resnet50_bucket(worker: int = 0, scale_seed: int = 3, data_seed_base: int = 100) -> Bucket:
    """ResNet-50-shaped bucket: conv/FC weights Laplace with per-tensor scale
    10^U(-5,-2); batch-norm and bias tensors Gaussian with sigma 1e-4.
    The per-tensor scales are shared by all workers; the values are not."""
    shapes = resnet50_shapes()
    scales = _log_uniform_scales(len(shapes), scale_seed)
    rng = _rng(data_seed_base + worker)
    sizes = [numel(s) for _, s in shapes]
    off = offsets_from_sizes(sizes)
    values = np.empty(int(off[-1]), dtype=np.float32)
    for t, (kind, _) in enumerate(shapes):
        n = sizes[t]
        if kind in ("conv", "fc_weight"):
            values[off[t] : off[t + 1]] = laplace(rng, n, float(scales[t]))
        else:
            values[off[t] : off[t + 1]] = gaussian(rng, n, 1e-4)
    return Bucket(values, off, [k for k, _ in shapes])


def vgg19_bucket(worker: int = 0, scale_seed: int = 3, data_seed_base: int = 100) -> Bucket:
    """VGG-19-shaped bucket: every tensor Student-t(nu=4) times a per-tensor
    scale 10^U(-5,-2) shared by all workers."""
    shapes = vgg19_shapes()
    scales = _log_uniform_scales(len(shapes), scale_seed)
    rng = _rng(data_seed_base + worker)
    sizes = [numel(s) for _, s in shapes]
    off = offsets_from_sizes(sizes)
    values = np.empty(int(off[-1]), dtype=np.float32)
    for t in range(len(shapes)):
        values[off[t] : off[t + 1]] = student_t(rng, sizes[t], 4.0, float(scales[t]))
    return Bucket(values, off, [k for k, _ in shapes])


def sweep_tensor(log2_n: int, seed: int = 7) -> Bucket:
    """Single Laplace(0, 1e-3) tensor of 2**log2_n elements for the roofline sweep."""
    v = laplace(_rng(seed), 1 << log2_n, 1e-3)
    return Bucket(v, offsets_from_sizes([v.size]), ["laplace"])
