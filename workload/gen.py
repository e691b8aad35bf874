"""Seeded synthetic request tables for the scheduler benchmarks.

This module only draws inputs: prompt lengths ``p`` and output lengths ``o`` per
request, clipped rounded log-normals.  It contains none of the scheduling
method's arithmetic and is imported by the tests, the benchmark and the smoke
check; neither the CPU oracle nor the CUDA library imports it.

Random numbers come from Philox4x32-10 (Salmon et al., "Parallel random
numbers: as easy as 1, 2, 3", SC'11), implemented here from its published
definition so that the bytes do not depend on the numpy version:

    counter = (request index, 0, 0, 0)      key = (seed mod 2^32, seed >> 32)

gives four 32-bit words per request.  Words 0,1 make the standard normal for
the prompt length and words 2,3 the one for the output length, each by the
Box-Muller cosine branch in float64:

    u1 = (w_a + 0.5) / 2^32   u2 = (w_b + 0.5) / 2^32
    z  = sqrt(-2 ln u1) * cos(2 pi u2)
    length = clip(rint(exp(ln(median) + sigma * z)), lo, hi)      (uint32)
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = np.uint64(0xFFFFFFFF)
_SH = np.uint64(32)


def philox4x32_10(counter0: np.ndarray, key0: int, key1: int):
    """Philox4x32 with 10 rounds for counters (counter0, 0, 0, 0); returns 4 uint32 arrays."""
    c0 = counter0.astype(np.uint64) & _MASK
    c1 = np.zeros_like(c0)
    c2 = np.zeros_like(c0)
    c3 = np.zeros_like(c0)
    k0 = key0 & 0xFFFFFFFF
    k1 = key1 & 0xFFFFFFFF
    for _ in range(10):
        prod0 = _M0 * c0
        prod1 = _M1 * c2
        hi0, lo0 = prod0 >> _SH, prod0 & _MASK
        hi1, lo1 = prod1 >> _SH, prod1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)), lo1, (hi0 ^ c3 ^ np.uint64(k1)), lo0
        k0 = (k0 + _W0) & 0xFFFFFFFF
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return (c0.astype(np.uint32), c1.astype(np.uint32), c2.astype(np.uint32), c3.astype(np.uint32))


def _normal(wa: np.ndarray, wb: np.ndarray) -> np.ndarray:
    u1 = (wa.astype(np.float64) + 0.5) / 4294967296.0
    u2 = (wb.astype(np.float64) + 0.5) / 4294967296.0
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


@dataclass(frozen=True)
class LengthDist:
    """clip(rint(lognormal(ln median, sigma)), lo, hi)."""
    median: float
    sigma: float
    lo: int
    hi: int

    def draw(self, z: np.ndarray) -> np.ndarray:
        x = np.rint(np.exp(np.log(self.median) + self.sigma * z))
        return np.clip(x, self.lo, self.hi).astype(np.uint32)


def instance_lengths(seed: int, n_req: int, dist_p: LengthDist, dist_o: LengthDist):
    """Prompt and output lengths (two uint32 arrays of n_req) of the instance with this seed."""
    idx = np.arange(n_req, dtype=np.uint64)
    w0, w1, w2, w3 = philox4x32_10(idx, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    return dist_p.draw(_normal(w0, w1)), dist_o.draw(_normal(w2, w3))


def estimated_outputs(seed: int, o: np.ndarray, sigma: float, lo: int, hi: int) -> np.ndarray:
    """Noisy estimates of the output lengths: clip(rint(o * exp(sigma * z)), lo, hi), z standard
    normal from the same generator under the key (seed mod 2^32, (seed >> 32) xor 0x45535431), words
    0 and 1.  sigma = 0 returns o clipped."""
    idx = np.arange(o.shape[0], dtype=np.uint64)
    w0, w1, _, _ = philox4x32_10(idx, seed & 0xFFFFFFFF, ((seed >> 32) ^ 0x45535431) & 0xFFFFFFFF)
    x = np.rint(o.astype(np.float64) * np.exp(sigma * _normal(w0, w1)))
    return np.clip(x, lo, hi).astype(np.uint32)


def batch_lengths(seeds, n_req: int, dist_p: LengthDist, dist_o: LengthDist):
    """Row-major [len(seeds)][n_req] uint32 tables p, o; row k is instance_lengths(seeds[k], ...)."""
    seeds = list(seeds)
    p = np.empty((len(seeds), n_req), dtype=np.uint32)
    o = np.empty((len(seeds), n_req), dtype=np.uint32)
    for k, s in enumerate(seeds):
        p[k], o[k] = instance_lengths(int(s), n_req, dist_p, dist_o)
    return p, o
