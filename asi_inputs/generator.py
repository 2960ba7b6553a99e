"""Seeded synthetic inputs for the ASI hot path.

This module only manufactures INPUT tensors (activations, output gradients,
previous-step factors).  It holds none of the method's arithmetic -- no
unfolding products, no subspace iteration, no weight gradient -- and is the
one module that both the CPU oracle's tests and the CUDA path's tests/bench
may import.

Recipe (stand-in for the paper's fine-tuning activations, which concentrate
their energy in the first few components of every mode and drift slowly from
step to step):

* generating core  G[k_1..k_n] = g * prod_m rho_m^{k_m},  g ~ N(0,1) i.i.d.,
  generating ranks R*_m (default min(D_m, 64));
* generating factors U*_m = Q factor of a seeded Gaussian D_m x R*_m matrix;
* signal = G x_1 U*_1 ... x_n U*_n, rescaled to unit RMS per element;
* A = signal + sigma * N(0,1), sigma = 1e-3; optional clip to [lo, hi]
  (post-ReLU6 activations);
* drift: every step the generating factors are rotated by exp(theta * K^),
  K = X - X^T with X ~ N(0,1), K^ = K / ||K||_2, theta = 0.01 rad, then
  re-orthonormalised; noise is fresh each step, the core is fixed;
* step-0 previous factors: the first r_m generating columns rotated by one
  extra drift step (a plausible "previous step" estimate);
* dY ~ N(0,1) / sqrt(number of summed positions), fresh each step.

Seeds: seed = base + 10000*config + 100*layer + step (see configs.py).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


def _orthonormal(rng, d, r):
    q, rr = np.linalg.qr(rng.standard_normal((d, r)))
    return q * np.sign(np.diag(rr))[None, :]


def _spectral_norm(K, rng, iters=40):
    x = rng.standard_normal(K.shape[1])
    x /= np.linalg.norm(x)
    s = 1.0
    for _ in range(iters):
        y = K @ x
        x = K.T @ y
        s = np.linalg.norm(x)
        x /= s
    return np.sqrt(s)


def _rotate(Ustar, rng, theta):
    """Apply exp(theta * K^) to the columns of Ustar (Taylor series, order 8),
    then re-orthonormalise."""
    d = Ustar.shape[0]
    X = rng.standard_normal((d, d))
    K = X - X.T
    nrm = _spectral_norm(K, rng) if d > 1 else 0.0
    if nrm == 0.0:                      # a mode of size one has nothing to rotate
        return Ustar.copy()
    K /= nrm
    term = Ustar.copy()
    out = Ustar.copy()
    for k in range(1, 9):
        term = (theta / k) * (K @ term)
        out += term
    q, rr = np.linalg.qr(out)
    return q * np.sign(np.diag(rr))[None, :]


def _expand(G, factors):
    T = G
    for m, Um in enumerate(factors):
        T = np.moveaxis(np.tensordot(Um, T, axes=([1], [m])), 0, m)
    return T


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to bfloat16, returned as float32 values that are
    exactly representable in bf16 (so the oracle can up-cast the very same
    numbers the GPU reads)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    rounded = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return rounded.astype(np.uint32).view(np.float32).reshape(x.shape)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of bf16-representable float32 values."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


@dataclass
class LayerStream:
    """Stateful generator of one layer's per-step inputs."""
    dims: tuple                      # activation shape (B,C,H,W) or (B,N,D)
    ranks: tuple                     # target ranks r_m
    dy_shape: tuple                  # shape of dY
    seed: int
    rho: tuple = None                # per-mode decay (default 0.7)
    gen_ranks: tuple = None          # generating ranks R*_m
    sigma: float = 1e-3
    theta: float = 0.01
    clip: tuple = None               # (lo, hi) or None
    bf16: bool = False               # round act and dY to bf16-representable values
    _step: int = field(default=0, init=False)

    def __post_init__(self):
        n = len(self.dims)
        if self.rho is None:
            self.rho = (0.7,) * n
        if self.gen_ranks is None:
            self.gen_ranks = tuple(min(d, 64) for d in self.dims)
        rng = np.random.default_rng(self.seed)
        G = rng.standard_normal(self.gen_ranks)
        for m in range(n):
            shape = [1] * n
            shape[m] = -1
            G = G * (self.rho[m] ** np.arange(self.gen_ranks[m])).reshape(shape)
        self._G = G
        self._Ustar = [_orthonormal(rng, d, r) for d, r in zip(self.dims, self.gen_ranks)]
        # previous-step estimate for step 0: leading generating columns, one drift step away
        self._U_prev0 = []
        for m in range(n):
            rot = _rotate(self._Ustar[m], rng, self.theta)
            self._U_prev0.append(np.ascontiguousarray(rot[:, :self.ranks[m]]))
        sig = _expand(self._G, self._Ustar)
        self._scale = 1.0 / np.sqrt(np.mean(sig * sig))

    def u_prev0(self):
        """fp32 previous-step factors handed to step 0."""
        return [u.astype(np.float32) for u in self._U_prev0]

    def skip(self, n: int):
        """Advances the stream by n steps without building the tensors: only the drift of the generating
        factors is replayed (each step seeds its own generator, so nothing else carries over)."""
        for _ in range(int(n)):
            rng = np.random.default_rng(self.seed + 1 + self._step)
            if self._step > 0:
                self._Ustar = [_rotate(u, rng, self.theta) for u in self._Ustar]
            self._step += 1

    def u_prev_now(self):
        """fp32 previous-step factors for the NEXT step: the leading generating columns as they stand,
        i.e. one drift step before the tensor that next() returns (the rule u_prev0() follows at step 0)."""
        return [np.ascontiguousarray(u[:, :r]).astype(np.float32) for u, r in zip(self._Ustar, self.ranks)]

    def next(self):
        """Returns (A, dY) of the next training step as float32 arrays
        (bf16-representable when ``bf16``); generating factors drift first for
        every step after the first."""
        rng = np.random.default_rng(self.seed + 1 + self._step)
        if self._step > 0:
            self._Ustar = [_rotate(u, rng, self.theta) for u in self._Ustar]
        A = _expand(self._G, self._Ustar) * self._scale
        A = A + self.sigma * rng.standard_normal(self.dims)
        if self.clip is not None:
            A = np.clip(A, self.clip[0], self.clip[1])
        nsum = int(np.prod(self.dy_shape)) // int(self.dy_shape[1 if len(self.dy_shape) == 4 else -1])
        dY = rng.standard_normal(self.dy_shape) / np.sqrt(nsum)
        self._step += 1
        A = A.astype(np.float32)
        dY = dY.astype(np.float32)
        if self.bf16:
            A, dY = round_to_bf16(A), round_to_bf16(dY)
        return A, dY
