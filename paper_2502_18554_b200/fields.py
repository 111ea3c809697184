"""Seeded synthetic inputs shaped like the paper's workloads (Table 5: fp32 scientific fields, flattened and fed
to a 1-D predictor; Section 4: messages of tens to hundreds of MB).  The paper's datasets are not redistributable
here, so these stand in for them.  This module holds none of the codec's arithmetic: it only makes arrays, in
float64, cast once to float32, and the same array feeds both the CPU oracle and the CUDA path.
"""
from __future__ import annotations

import numpy as np

__all__ = ["smooth_1d", "fourier_field_3d", "gradient_like", "rank_fields", "on_grid_ranks"]


def smooth_1d(n: int, seed: int = 0, chunk: int = 1 << 22) -> np.ndarray:
    """Sum of 3 sinusoids (amplitude U(0.5,2), period U(1e3,1e5) samples, phase U(0,2pi)) plus N(0, sigma=1e-3)."""
    rng = np.random.default_rng(seed)
    amp = rng.uniform(0.5, 2.0, 3)
    period = rng.uniform(1e3, 1e5, 3)
    phase = rng.uniform(0.0, 2.0 * np.pi, 3)
    out = np.empty(n, np.float32)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        i = np.arange(lo, hi, dtype=np.float64)
        v = np.zeros(hi - lo, np.float64)
        for a, p, ph in zip(amp, period, phase):
            v += a * np.sin(2.0 * np.pi * i / p + ph)
        v += rng.normal(0.0, 1e-3, hi - lo)
        out[lo:hi] = v
    return out


def fourier_field_3d(side: int = 256, seed: int = 1, modes: int = 64, kmax: int = 16, noise: float = 1e-4) -> np.ndarray:
    """side^3 Gaussian-random-field stand-in: `modes` cosine modes with integer wavevectors 1 <= |k| <= kmax,
    amplitude |k|^-2, random phases, plus N(0, sigma=noise); flattened row-major."""
    rng = np.random.default_rng(seed)
    spec = np.zeros((side, side, side), np.complex128)
    placed = 0
    while placed < modes:
        k = rng.integers(-kmax, kmax + 1, 3)
        kn = float(np.sqrt((k * k).sum()))
        if kn < 1.0 or kn > kmax:
            continue
        phase = rng.uniform(0.0, 2.0 * np.pi)
        amp = kn ** -2.0
        # amp*cos(k.x + phase) = Re(amp e^{i phase} e^{i k.x}); ifftn carries a 1/side^3 factor
        spec[k[0] % side, k[1] % side, k[2] % side] += amp * np.exp(1j * phase) * side ** 3
        placed += 1
    field = np.fft.ifftn(spec).real
    del spec
    field += rng.normal(0.0, noise, field.shape)
    return np.ascontiguousarray(field.reshape(-1), dtype=np.float32)


def gradient_like(n: int, seed: int = 3, chunk: int = 1 << 24) -> np.ndarray:
    """Laplace(0, b=1e-3) with 10 % exact zeros and 0.1 % outliers drawn from N(0, sigma=1e-1)."""
    rng = np.random.default_rng(seed)
    out = np.empty(n, np.float32)
    for lo in range(0, n, chunk):
        m = min(n, lo + chunk) - lo
        v = rng.laplace(0.0, 1e-3, m)
        u = rng.random(m)
        v[u < 0.10] = 0.0
        sel = u > 0.999
        v[sel] = rng.normal(0.0, 1e-1, int(sel.sum()))
        out[lo:lo + m] = v
    return out


def rank_fields(nranks: int, n: int, base_seed: int = 100, kind: str = "fourier") -> list[np.ndarray]:
    """One differently seeded field per emulated rank (seed = base_seed + rank)."""
    fields = []
    for r in range(nranks):
        if kind == "fourier":
            side = round(n ** (1.0 / 3.0))
            if side ** 3 != n:
                raise ValueError("fourier rank fields need a cubic element count")
            fields.append(fourier_field_3d(side, seed=base_seed + r))
        elif kind == "smooth":
            fields.append(smooth_1d(n, seed=base_seed + r))
        else:
            raise ValueError(kind)
    return fields


def on_grid_ranks(nranks: int, n: int, step: float, seed: int = 7, kmax: int = 1000) -> list[np.ndarray]:
    """Rank buffers whose values are small integer multiples of `step` (a power of two), so that every
    quantisation and every partial sum is exact in fp32: the lossless special case of the ring Allreduce."""
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(nranks):
        walk = np.cumsum(rng.integers(-3, 4, n))
        walk = np.clip(walk, -kmax, kmax)
        out.append((walk.astype(np.float64) * step).astype(np.float32))
    return out
