"""Seeded synthetic series standing in for the paper's benchmark windows.

Every recipe returns ``[B, ctx_len + H]`` float32, z-normalised per series over
its whole length: seasonal sinusoids + linear trend + AR(1) noise, optionally
cumulative level shifts and isolated spikes.  The tail of length H is ground
truth (unused by the decoding path).
"""
from __future__ import annotations

import numpy as np
from scipy.signal import lfilter

from .configs import Workload


def _ar1(rng, B, n, phi, sigma):
    eps = rng.standard_normal((B, n)) * sigma
    out = np.empty((B, n))
    phi = np.broadcast_to(np.asarray(phi, dtype=np.float64), (B,))
    for b in range(B):
        out[b] = lfilter([1.0], [1.0, -phi[b]], eps[b])
    return out


def _znorm(y):
    return (y - y.mean(axis=1, keepdims=True)) / y.std(axis=1, keepdims=True)


def make_series(wl: Workload, batch: int | None = None) -> np.ndarray:
    B = wl.batch if batch is None else batch
    n = wl.ctx_len + wl.horizon
    rng = np.random.default_rng([wl.series_seed, 0x5e71])
    t = np.arange(n, dtype=np.float64)[None, :]
    recipe = wl.series_recipe
    if recipe == "c0":
        y = np.sin(2 * np.pi * t / 24) + 0.5 * np.sin(2 * np.pi * t / 168) + 0.01 * t
        y = np.repeat(y, B, axis=0) + _ar1(rng, B, n, 0.8, 0.1)
    elif recipe in ("c1", "c2"):
        period = rng.choice([12.0, 24.0, 48.0], size=(B, 1))
        slope = rng.uniform(-0.02, 0.02, size=(B, 1))
        phi = rng.uniform(0.5, 0.95, size=B)
        y = np.sin(2 * np.pi * t / period) + 0.5 * np.sin(2 * np.pi * t / 168) + slope * t
        y = y + _ar1(rng, B, n, phi, 0.1)
        if recipe == "c2":
            jumps = (rng.random((B, n)) < 1.0 / 500.0) * rng.normal(0.0, 2.0, size=(B, n))
            y = y + np.cumsum(jumps, axis=1)
    elif recipe == "c4":
        slope = rng.uniform(-0.002, 0.002, size=(B, 1))
        phi = rng.uniform(0.5, 0.95, size=B)
        y = (np.sin(2 * np.pi * t / 24) + 0.5 * np.sin(2 * np.pi * t / 168)
             + 0.25 * np.sin(2 * np.pi * t / 720) + slope * t)
        y = y + _ar1(rng, B, n, phi, 0.1)
        jumps = (rng.random((B, n)) < 1.0 / 500.0) * rng.normal(0.0, 2.0, size=(B, n))
        y = y + np.cumsum(jumps, axis=1)
        y = y + (rng.random((B, n)) < 1.0 / 1000.0) * rng.normal(0.0, 5.0, size=(B, n))
    else:
        raise ValueError(f"unknown series recipe {recipe!r}")
    return _znorm(y).astype(np.float32)
