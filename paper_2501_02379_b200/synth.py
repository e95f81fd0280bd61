"""Seeded synthetic inputs: FNO-shaped complex gradients and weights.

This module only *generates inputs* (numpy, CPU).  It holds none of the
optimizer's arithmetic and imports neither the CUDA binding nor the CPU
oracle; both sides of a parity test receive the very same bytes produced
here.

A gradient is built the way the paper describes FNO spectral-weight
gradients (Section 2.2, "Robust decomposition of gradients"): a tensor of low
mode-wise (Tucker) rank, plus a few gross outliers, plus dense noise:

    G_t = [[C_t; A_1 .. A_N]] + outliers_t + noise_t

* A_n: orthonormal I_n x r_n factors (Q of a QR of a complex normal matrix),
  fixed for the whole run of a tensor.
* C_t = Cbar + 0.5 E_t, Cbar and E_t complex standard normal (re, im ~ N(0,1)).
* outliers_t[p] = s * sigma_sig * u_p * (1 + 0.1 xi_{t,p}) on a fixed set P of
  flat positions with fixed unit phases u_p; sigma_sig = rms |signal at t=0|.
* noise_t: i.i.d. per real/imaginary part, family and scale per workload.

Every random draw comes from a Philox stream keyed by (seed, step, part), so
any step's gradient can be regenerated on its own.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional, Tuple

import numpy as np

BASE_SEED = 250102379


@dataclasses.dataclass(frozen=True)
class Workload:
    """One named workload: tensor shape, compression settings, input recipe."""

    name: str
    cfg_id: int
    shape: Tuple[int, ...]
    ranks: Tuple[int, ...]            # Tucker ranks r_n used by the optimizer
    rho: Tuple[int, int]              # sparsity as an exact fraction (num, den)
    T: int                            # refresh period
    steps: int
    n_tensors: int = 1
    signal_ranks: Optional[Tuple[int, ...]] = None   # planted ranks (default = ranks)
    outlier_frac: Tuple[int, int] = (0, 1)
    outliers_equal_k: bool = False    # |P| = k exactly (workload 1)
    outlier_scale: float = 0.0
    noise: str = "normal"             # normal | student_t2 | laplace
    noise_scale: float = 0.0          # std (normal), scale b (laplace), x sigma_sig (student)
    half_storage: bool = False        # W, G stored as interleaved fp16 pairs
    bf16_storage: bool = False        # ... or as interleaved bfloat16 pairs
    lr: float = 1e-3

    @property
    def numel(self) -> int:
        return int(np.prod(self.shape, dtype=np.int64))

    @property
    def k(self) -> int:
        num, den = self.rho
        return -((-self.numel * num) // den)       # exact ceil(rho * I)

    @property
    def n_outliers(self) -> int:
        if self.outliers_equal_k:
            return self.k
        num, den = self.outlier_frac
        return -((-self.numel * num) // den)

    @property
    def planted_ranks(self) -> Tuple[int, ...]:
        return self.signal_ranks if self.signal_ranks is not None else self.ranks


WORKLOADS: Dict[str, Workload] = {
    w.name: w
    for w in [
        # tiny cases for quick tests (not from the benchmark list)
        Workload("tiny4", 90, (6, 5, 4, 3), (3, 2, 2, 2), (1, 20), 3, 7,
                 outliers_equal_k=True, outlier_scale=20.0, noise_scale=0.01),
        Workload("small4", 91, (12, 10, 8, 5), (4, 3, 3, 2), (3, 100), 4, 9,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise_scale=0.02),
        Workload("small5", 92, (6, 5, 4, 4, 3), (3, 2, 2, 2, 2), (1, 50), 3, 7,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise="laplace", noise_scale=0.1),
        Workload("ragged4", 93, (20, 12, 24, 13), (5, 4, 6, 4), (1, 40), 4, 9,
                 outlier_frac=(1, 200), outlier_scale=30.0, noise_scale=0.03),
        # shapes that reach the tensor-core streaming kernels in their corner cases: a 3-way tensor (no
        # mode product outside the fused first-mode launch) and a slab count that leaves the last group of
        # slabs partly empty
        Workload("small3", 94, (12, 16, 9), (4, 4, 3), (1, 40), 3, 7,
                 outlier_frac=(1, 200), outlier_scale=25.0, noise_scale=0.02),
        Workload("odd4", 95, (7, 9, 16, 9), (3, 4, 4, 3), (1, 50), 3, 7,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise="laplace", noise_scale=0.05),
        Workload("odd32", 96, (5, 7, 32, 17), (3, 3, 8, 5), (1, 25), 3, 5,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise_scale=0.05),
        # a 5-way tensor whose middle mode product has many small slices (the shared-memory fp32 product kernel)
        Workload("small5b", 97, (8, 9, 6, 16, 9), (3, 3, 3, 4, 3), (1, 50), 3, 5,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise_scale=0.05),
        # shapes that reach the kernels only the largest configuration would otherwise run: 65-entry rows of a
        # 128-row slab stored as fp16 with trailing ranks (32, 16); a leading extent whose Gram matrix is too large
        # for the eigensolver's shared-memory path (161..256) and one beyond its rotation-log path (> 256, which
        # also takes the first mode out of the fused launch); a trailing extent (19) whose tile count is not built in
        Workload("half65", 98, (3, 4, 128, 65), (2, 3, 32, 16), (1, 100), 3, 5,
                 outlier_frac=(1, 200), outlier_scale=20.0, noise_scale=0.02, half_storage=True),
        Workload("lead200", 99, (200, 6, 8, 5), (4, 3, 3, 2), (1, 50), 3, 5,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise_scale=0.02),
        Workload("lead300", 100, (300, 5, 8, 5), (4, 3, 3, 2), (1, 50), 3, 5,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise_scale=0.02),
        Workload("tail19", 101, (5, 6, 16, 19), (3, 3, 4, 3), (1, 50), 3, 5,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise_scale=0.05),
        # leading modes with long contiguous rows and 64..256 entries (the tcgen05 Gram kernel): two 128-row tiles of
        # the Gram matrix, fp16 storage with a row count that is not a multiple of 16, and an odd row count
        Workload("gram144", 103, (144, 40, 32, 17), (8, 6, 6, 4), (1, 50), 3, 5,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise_scale=0.02),
        Workload("gram96h", 104, (96, 72, 32, 17), (8, 6, 6, 4), (1, 100), 3, 5,
                 outlier_frac=(1, 200), outlier_scale=20.0, noise_scale=0.02, half_storage=True),
        Workload("gram75", 105, (75, 64, 32, 16), (6, 8, 6, 4), (1, 50), 3, 5,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise_scale=0.02),
        # the matrix case (N = 2)
        Workload("mat2", 102, (96, 80), (12, 10), (1, 50), 3, 7,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise_scale=0.02),
        # the five benchmark configurations
        Workload("cfg1", 1, (32, 32, 16, 9), (8, 8, 4, 3), (1, 100), 5, 20,
                 outliers_equal_k=True, outlier_scale=20.0, noise_scale=0.01, lr=1e-3),
        Workload("cfg2", 2, (64, 64, 32, 17), (16, 16, 8, 5), (5, 100), 50, 200, n_tensors=4,
                 noise="student_t2", noise_scale=0.05),
        Workload("cfg3", 3, (128, 128, 64, 33), (32, 32, 16, 8), (25, 1000), 100, 500,
                 outlier_frac=(5, 1000), outlier_scale=50.0, noise_scale=0.05),
        Workload("cfg4", 4, (64, 64, 32, 32, 17), (16, 16, 8, 8, 5), (2, 100), 100, 300,
                 outlier_frac=(1, 100), outlier_scale=20.0, noise="laplace", noise_scale=0.1),
        Workload("cfg5", 5, (256, 256, 128, 65), (64, 64, 32, 16), (1, 100), 200, 100,
                 outlier_frac=(5, 1000), outlier_scale=30.0, noise_scale=0.02, half_storage=True),
        # the same slabs, ranks and storage with smaller leading extents (0.3 GB per tensor): the case the
        # profiler captures of the largest configuration's kernels are taken on
        Workload("cfg5p", 5, (96, 96, 128, 65), (64, 64, 32, 16), (1, 100), 200, 100,
                 outlier_frac=(5, 1000), outlier_scale=30.0, noise_scale=0.02, half_storage=True),
    ]
}


def _rng(seed: int, step: int, part: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=seed, counter=[step, part, 0, 0]))


def _cnormal(rng: np.random.Generator, shape, scale: float = 1.0) -> np.ndarray:
    """Complex normal: re, im i.i.d. N(0, scale^2); complex64."""
    x = rng.standard_normal(tuple(shape) + (2,), dtype=np.float32)
    if scale != 1.0:
        x *= np.float32(scale)
    return x.view(np.complex64)[..., 0]


def _expand(core: np.ndarray, factors) -> np.ndarray:
    """[[core; A_1..A_N]] in complex64 (input synthesis only)."""
    x = core
    for n, a in enumerate(factors):
        x = np.moveaxis(np.tensordot(a, x, axes=([1], [n])), 0, n)
    return np.ascontiguousarray(x)


class GradientSource:
    """Deterministic gradient / weight generator for one tensor of a workload."""

    def __init__(self, wl: Workload, tensor_id: int = 0):
        self.wl = wl
        self.seed = BASE_SEED + 1000 * wl.cfg_id + tensor_id
        shape, pr = wl.shape, wl.planted_ranks
        r0 = _rng(self.seed, 0, 1)
        self.factors = []
        for i_n, r_n in zip(shape, pr):
            q, _ = np.linalg.qr(_cnormal(r0, (i_n, r_n)).astype(np.complex128))
            self.factors.append(np.ascontiguousarray(q.astype(np.complex64)))
        self.core_mean = _cnormal(r0, pr)
        c0 = self._core(0)
        # factors are orthonormal, so ||signal_0||_F = ||C_0||_F
        self.sigma_sig = float(np.sqrt(np.sum(np.abs(c0.astype(np.complex128)) ** 2) / wl.numel))
        n_out = wl.n_outliers
        if n_out > 0 and wl.outlier_scale > 0.0:
            self.out_pos = self._distinct_positions(n_out)
            ph = _rng(self.seed, 0, 3).uniform(0.0, 2.0 * math.pi, size=n_out)
            self.out_phase = np.exp(1j * ph).astype(np.complex64)
        else:
            self.out_pos = np.zeros(0, dtype=np.int64)
            self.out_phase = np.zeros(0, dtype=np.complex64)

    def _distinct_positions(self, n: int) -> np.ndarray:
        rng = _rng(self.seed, 0, 2)
        total = self.wl.numel
        pos = np.unique(rng.integers(0, total, size=n, dtype=np.int64))
        while pos.size < n:
            extra = rng.integers(0, total, size=2 * (n - pos.size) + 16, dtype=np.int64)
            pos = np.unique(np.concatenate([pos, extra]))
        if pos.size > n:
            drop = rng.choice(pos.size, size=pos.size - n, replace=False)
            pos = np.delete(pos, drop)
        return pos

    def _core(self, step: int) -> np.ndarray:
        e = _cnormal(_rng(self.seed, step, 10), self.wl.planted_ranks)
        return (self.core_mean + np.float32(0.5) * e).astype(np.complex64)

    def signal(self, step: int) -> np.ndarray:
        return _expand(self._core(step), self.factors)

    def weight(self) -> np.ndarray:
        """W_0 ~ complex N(0, 0.02^2), complex64."""
        return _cnormal(_rng(self.seed, 0, 4), self.wl.shape, 0.02)

    def gradient(self, step: int) -> np.ndarray:
        """G_t as complex64, C-contiguous, shape wl.shape."""
        wl = self.wl
        g = self.signal(step)
        flat = g.reshape(-1)
        if wl.noise_scale > 0.0:
            rng = _rng(self.seed, step, 11)
            if wl.noise == "normal":
                chunk = 1 << 24
                fv = flat.view(np.float32)
                for s in range(0, fv.size, chunk):
                    e = min(fv.size, s + chunk)
                    fv[s:e] += np.float32(wl.noise_scale) * rng.standard_normal(e - s, dtype=np.float32)
            elif wl.noise == "laplace":
                fv = flat.view(np.float32)
                chunk = 1 << 24
                for s in range(0, fv.size, chunk):
                    e = min(fv.size, s + chunk)
                    fv[s:e] += rng.laplace(0.0, wl.noise_scale, size=e - s).astype(np.float32)
            elif wl.noise == "student_t2":
                fv = flat.view(np.float32)
                sc = wl.noise_scale * self.sigma_sig
                fv += (sc * rng.standard_t(2.0, size=fv.size)).astype(np.float32)
            else:
                raise ValueError(wl.noise)
        if self.out_pos.size:
            xi = _rng(self.seed, step, 12).standard_normal(self.out_pos.size, dtype=np.float32)
            amp = np.float32(wl.outlier_scale * self.sigma_sig) * (np.float32(1.0) + np.float32(0.1) * xi)
            flat[self.out_pos] += self.out_phase * amp
        return g


def to_half_pairs(x: np.ndarray) -> np.ndarray:
    """complex64 -> interleaved IEEE fp16 (re, im) pairs, shape (..., 2)."""
    return np.ascontiguousarray(x).view(np.float32).reshape(x.shape + (2,)).astype(np.float16)


def from_half_pairs(h: np.ndarray) -> np.ndarray:
    """interleaved fp16 pairs (..., 2) -> complex64 (exact widening)."""
    return np.ascontiguousarray(h.astype(np.float32)).view(np.complex64)[..., 0]


def to_bf16_pairs(x: np.ndarray) -> np.ndarray:
    """complex64 -> interleaved bfloat16 (re, im) pairs as uint16 bit patterns, shape (..., 2); nearest, ties to even."""
    u = np.ascontiguousarray(x).view(np.float32).reshape(x.shape + (2,)).view(np.uint32).astype(np.uint64)
    bias = ((u >> np.uint64(16)) & np.uint64(1)) + np.uint64(0x7FFF)
    return ((u + bias) >> np.uint64(16)).astype(np.uint16)


def from_bf16_pairs(b: np.ndarray) -> np.ndarray:
    """interleaved bfloat16 bit patterns (..., 2) -> complex64 (exact widening)."""
    return np.ascontiguousarray((b.astype(np.uint32) << np.uint32(16)).view(np.float32)).view(np.complex64)[..., 0]


def quantised_ties(shape, levels: int, seed: int) -> np.ndarray:
    """Tie-heavy complex64 tensor: re, im on a small integer grid (many equal |g|^2)."""
    rng = _rng(seed, 0, 20)
    x = rng.integers(-levels, levels + 1, size=tuple(shape) + (2,)).astype(np.float32)
    return x.view(np.complex64)[..., 0]
