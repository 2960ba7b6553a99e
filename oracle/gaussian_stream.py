"""Counter-based Gaussian test matrices for the cold start (Algorithm 1, t = 0: "V ~ N(0, 1)") -- the oracle's
side.  Test infrastructure only: the product package never imports this file.

The paper fixes no generator.  Both sides of the parity tests implement the same published one so that a seed
alone defines Omega_m:

  * Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11): a
    128-bit counter and a 64-bit key give four 32-bit words after ten rounds of
        (c0, c1, c2, c3) <- (hi(M1 c2) ^ c1 ^ k0,  lo(M1 c2),  hi(M0 c0) ^ c3 ^ k1,  lo(M0 c0)),
    the key advancing by the Weyl constants (W0, W1) between rounds.
  * key = the 64-bit seed (low word, high word); counter = (g mod 2^32, g div 2^32, stream, 0) where g is the
    index of a group of four consecutive values and `stream` is the mode m.
  * words -> uniforms in (0, 1): u = ((x >> 9) + 0.5) 2^-23 (24 significant bits: exact in fp32);
    Box-Muller on the pairs (x0, x1) and (x2, x3): z = sqrt(-2 ln u_a) (cos, sin)(2 pi u_b).
  * Omega_m[e] for the row-major element index e is value e mod 4 of group e div 4.

Here the transform runs in fp64 from the exact uniforms; the CUDA side runs it in fp32, so the two agree to fp32
rounding of log, sqrt, sin and cos (a few 1e-7 relative to |z| <= 6).  The words themselves are compared bit for
bit.  Pins: tests/test_oracle_gaussian_stream.py (the generator's published known-answer vectors, the Box-Muller
closed form at hand-picked uniforms, moments)."""
from __future__ import annotations

import numpy as np

M0 = np.uint64(0xD2511F53)
M1 = np.uint64(0xCD9E8D57)
W0 = 0x9E3779B9
W1 = 0xBB67AE85
MASK = np.uint64(0xFFFFFFFF)


def philox4x32_10(counter, key):
    """counter: integer array [..., 4], key: integer array [..., 2] (32-bit words).  Returns uint32 [..., 4]."""
    c = np.asarray(counter, dtype=np.uint64) & MASK
    k = np.asarray(key, dtype=np.uint64) & MASK
    c0, c1, c2, c3 = (c[..., i].copy() for i in range(4))
    k0, k1 = k[..., 0].copy(), k[..., 1].copy()
    for _ in range(10):
        p0 = M0 * c0                       # 32 x 32 -> 64 bits, exact in uint64
        p1 = M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & MASK
        hi1, lo1 = p1 >> np.uint64(32), p1 & MASK
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + np.uint64(W0)) & MASK
        k1 = (k1 + np.uint64(W1)) & MASK
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def words(seed: int, stream: int, n_groups: int) -> np.ndarray:
    """The first n_groups groups of four words of (seed, stream): uint32 [n_groups, 4]."""
    g = np.arange(n_groups, dtype=np.uint64)
    ctr = np.stack([g & MASK, g >> np.uint64(32), np.full_like(g, stream), np.zeros_like(g)], axis=-1)
    key = np.array([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF], dtype=np.uint64)
    return philox4x32_10(ctr, np.broadcast_to(key, (n_groups, 2)))


def uniform_from_word(x) -> np.ndarray:
    return ((np.asarray(x, dtype=np.uint64) >> np.uint64(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def box_muller(ua, ub):
    rad = np.sqrt(-2.0 * np.log(ua))
    return rad * np.cos(2.0 * np.pi * ub), rad * np.sin(2.0 * np.pi * ub)


def gaussian(seed: int, stream: int, n: int) -> np.ndarray:
    """The first n values of the N(0, 1) stream (seed, stream), fp64."""
    ng = (n + 3) // 4
    u = uniform_from_word(words(seed, stream, ng))
    z0, z1 = box_muller(u[:, 0], u[:, 1])
    z2, z3 = box_muller(u[:, 2], u[:, 3])
    return np.stack([z0, z1, z2, z3], axis=-1).reshape(-1)[:n]


def omega_matrices(seed: int, dims, ranks) -> list:
    """Omega_m [b_m x r_m], b_m = prod of the other modes' sizes, for every mode m (stream = m)."""
    total = int(np.prod(dims))
    out = []
    for m, (d, r) in enumerate(zip(dims, ranks)):
        b = total // int(d)
        out.append(gaussian(seed, m, b * int(r)).reshape(b, int(r)))
    return out
