"""Oracle, part 3: counter-based random numbers for the synthetic gradients (TEST INFRASTRUCTURE ONLY).

Philox4x32-10 as defined by Salmon, Moraes, Dror and Shaw, "Parallel random numbers: as easy as
1, 2, 3" (SC'11): a 4x32-bit counter, a 2x32-bit key, ten rounds of two 32x32->64 multiplications
with the constants below, the key bumped by the Weyl constants between rounds.  Normals by the
Box-Muller transform on 23-bit uniforms u = (n + 1/2) * 2^-23, which float32 holds exactly.

Synthetic gradient of worker i at iteration k for parameter p (stands in for back-propagation):
    counter = (p // 4, i, k, 6), key = (seed mod 2^32, seed div 2^32)
    (r0, r1, r2, r3) = philox(counter, key)
    z[4q+0], z[4q+1] = BoxMuller(r0, r1);  z[4q+2], z[4q+3] = BoxMuller(r2, r3)
    G = sigma * z
"""
from __future__ import annotations

import numpy as np

M0 = np.uint64(0xD2511F53)
M1 = np.uint64(0xCD9E8D57)
W0 = 0x9E3779B9
W1 = 0xBB67AE85
MASK = np.uint64(0xFFFFFFFF)
GRAD_STREAM = 6


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Vectorised over numpy arrays of counters; returns four uint32 arrays."""
    c0 = np.asarray(c0, np.uint64) & MASK
    c1 = np.asarray(c1, np.uint64) & MASK
    c2 = np.asarray(c2, np.uint64) & MASK
    c3 = np.asarray(c3, np.uint64) & MASK
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for r in range(10):
        p0 = M0 * c0                      # 64-bit products of 32-bit values
        p1 = M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & MASK
        hi1, lo1 = p1 >> np.uint64(32), p1 & MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)), lo1, (hi0 ^ c3 ^ np.uint64(k1)), lo0
        k0 = (k0 + W0) & 0xFFFFFFFF
        k1 = (k1 + W1) & 0xFFFFFFFF
    return (c0.astype(np.uint32), c1.astype(np.uint32), c2.astype(np.uint32), c3.astype(np.uint32))


def _uniform23(r):
    return ((r >> np.uint32(9)).astype(np.float64) + 0.5) * (2.0 ** -23)


def box_muller(ra, rb):
    u1 = _uniform23(ra)
    u2 = _uniform23(rb)
    rad = np.sqrt(-2.0 * np.log(u1))
    ang = 2.0 * np.pi * u2
    return rad * np.cos(ang), rad * np.sin(ang)


def synthetic_gradient(seed: int, worker: int, level: int, cols: np.ndarray, sigma: float) -> np.ndarray:
    """G[worker][cols] at iteration `level`, float64."""
    cols = np.asarray(cols, np.int64)
    q = cols // 4
    e = cols % 4
    r0, r1, r2, r3 = philox4x32_10(q, np.full_like(q, worker), np.full_like(q, level),
                                   np.full_like(q, GRAD_STREAM), seed & 0xFFFFFFFF, seed >> 32)
    z0, z1 = box_muller(r0, r1)
    z2, z3 = box_muller(r2, r3)
    z = np.where(e == 0, z0, np.where(e == 1, z1, np.where(e == 2, z2, z3)))
    return sigma * z
