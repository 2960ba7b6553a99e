"""fp64 CPU oracle for the ASI (Activation Subspace Iteration) hot path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
CUDA library must compute.  It shares no code with the CUDA path and must never
be imported by the product package; only the test-suite, the smoke check and
the CPU-baseline leg of the benchmark may call it.

Everything is float64 NumPy.  Library primitives used as single steps:
``np.tensordot`` / ``@`` (dense contraction) and ``np.linalg.eigvalsh`` (only in
the HOSVD energy-rank helper).  There is no blocking, fusion or reordering
beyond what the cited passage states.

Parity pins (see tests/test_oracle_*.py): every function below is pinned by
brute-force definitions on tiny tensors, closed forms, invariants and the
values printed in the paper's ImageNet table.  The one thing the paper does
not fix is a printed numeric output of Algorithm 1 on given data; that single
item is "parity unpinned" -- agreement there rests on the invariants
(exactness at full rank, exact recovery of an exactly low-rank tensor,
convergence to the truncated-HOSVD subspace).

Notation follows the paper: activation A in R^{B x C x H x W} (or B x N x D for
token layers), mode-m unfolding A_m in R^{a_m x b_m}, factors U_m in
R^{a_m x r_m}, core S in R^{r_1 x ... x r_n}.
"""
from __future__ import annotations

import numpy as np


class RankDeficientError(ArithmeticError):
    """Raised when Orthogonalize meets a (numerically) dependent column."""


# --------------------------------------------------------------------------
# Tensor algebra primitives (Sec. 3.2)
# --------------------------------------------------------------------------
def unfold(T: np.ndarray, m: int) -> np.ndarray:
    """Mode-m unfolding A_m in R^{a_m x b_m}, a_m = D_m, b_m = prod of the other
    dimensions (Sec. 3.2, first paragraph).  Columns are ordered with the
    remaining modes in increasing order, last mode fastest; every quantity
    built from A_m A_m^T is independent of that column order."""
    T = np.asarray(T, dtype=np.float64)
    return np.moveaxis(T, m, 0).reshape(T.shape[m], -1)


def mode_product(G: np.ndarray, Bmat: np.ndarray, m: int) -> np.ndarray:
    """m-mode product R = G x_m B with B in R^{Q x P_m} (Sec. 3.2, the display
    after the Tucker form; the printed subscript of g is garbled, the reading
    is  R[.., q, ..] = sum_{p_m} G[.., p_m, ..] * B[q, p_m])."""
    G = np.asarray(G, dtype=np.float64)
    Bmat = np.asarray(Bmat, dtype=np.float64)
    if Bmat.ndim != 2 or Bmat.shape[1] != G.shape[m]:
        raise ValueError("mode_product: B must be Q x P_m")
    R = np.tensordot(Bmat, G, axes=([1], [m]))  # [Q, other modes...]
    return np.moveaxis(R, 0, m)


def orthogonalize(P: np.ndarray, rel_tol: float = 1e-12) -> np.ndarray:
    """Orthogonalize(P) of Algorithm 1: the result of Gram-Schmidt on the
    columns of P in exact arithmetic, i.e. the thin-QR factor Q whose R has a
    positive diagonal.  Computed by Householder reflections (numerically
    stable), then column signs are fixed so that diag(Q^T P) > 0.

    Raises RankDeficientError when a pivot column norm falls below
    rel_tol * ||P||_F (a dependent column has no Gram-Schmidt direction)."""
    P = np.array(P, dtype=np.float64, copy=True)
    a, r = P.shape
    if r > a:
        raise ValueError("orthogonalize: need r <= a")
    scale = np.linalg.norm(P)
    if scale == 0.0:
        raise RankDeficientError("zero matrix")
    R = P
    vs = []
    diag_sign = np.ones(r)
    for j in range(r):
        x = R[j:, j].copy()
        nx = np.sqrt(np.sum(x * x))
        if nx < rel_tol * scale:
            raise RankDeficientError(f"column {j}: pivot norm {nx:.3e}")
        alpha = -nx if x[0] >= 0.0 else nx      # R[j, j] after the reflection
        v = x
        v[0] -= alpha
        nv = np.sqrt(np.sum(v * v))
        v = v / nv
        vs.append(v)
        R[j:, j:] -= 2.0 * np.outer(v, v @ R[j:, j:])
        diag_sign[j] = 1.0 if alpha > 0.0 else -1.0
    # Q = H_0 H_1 ... H_{r-1} [I_r; 0]
    Q = np.zeros((a, r))
    Q[:r, :r] = np.eye(r)
    for j in reversed(range(r)):
        v = vs[j]
        Q[j:, :] -= 2.0 * np.outer(v, v @ Q[j:, :])
    return Q * diag_sign[None, :]


# --------------------------------------------------------------------------
# Algorithm 1 (ASI)
# --------------------------------------------------------------------------
def _check_ranks(shape, ranks):
    n = int(np.prod(shape))
    for m, (d, r) in enumerate(zip(shape, ranks)):
        if not (1 <= r <= min(d, n // d)):
            raise ValueError(f"rank {r} of mode {m} outside [1, min(a_m, b_m)]")


def subspace_step(A: np.ndarray, m: int, U_prev_m: np.ndarray) -> np.ndarray:
    """One warm-started subspace iteration on mode m (Algorithm 1, loop body,
    branch t > 0):  V = A_m^T U_m^{(t-1)};  U_m^{(t)} = Orthogonalize(A_m V).
    The right-hand U carries the previous step's superscript (the printed
    algorithm shows the same superscript on both sides)."""
    Am = unfold(A, m)
    V = Am.T @ np.asarray(U_prev_m, dtype=np.float64)     # b_m x r_m
    P = Am @ V                                            # a_m x r_m
    return orthogonalize(P)


def cold_start_step(A: np.ndarray, m: int, Omega_m: np.ndarray) -> np.ndarray:
    """Algorithm 1, branch t = 0:  V is an i.i.d. N(0,1) matrix of size
    b_m x r_m (passed in as Omega_m so both sides of a comparison can share
    it);  U_m^{(0)} = Orthogonalize(A_m V)."""
    Am = unfold(A, m)
    Omega_m = np.asarray(Omega_m, dtype=np.float64)
    if Omega_m.shape[0] != Am.shape[1]:
        raise ValueError("Omega must be b_m x r_m")
    return orthogonalize(Am @ Omega_m)


def core_tensor(A: np.ndarray, U: list) -> np.ndarray:
    """S = A x_1 U_1^T x_2 U_2^T ... x_n U_n^T (Algorithm 1, the core update,
    with U_m^T: the printed S x_m U_m does not type-check against the
    definition of the m-mode product, which needs a Q x P_m = r_m x a_m
    matrix)."""
    S = np.asarray(A, dtype=np.float64)
    for m, Um in enumerate(U):
        S = mode_product(S, np.asarray(Um, dtype=np.float64).T, m)
    return S


def asi_compress(A: np.ndarray, U_prev: list, ranks=None):
    """Algorithm 1 for t > 0.  Every mode unfolds the ORIGINAL activation (the
    algorithm says "unfold A^{(t)}", not the running core), so the modes are
    independent.  Returns (S, [U_1..U_n])."""
    A = np.asarray(A, dtype=np.float64)
    if len(U_prev) != A.ndim:
        raise ValueError("one previous factor per mode")
    if ranks is None:
        ranks = [u.shape[1] for u in U_prev]
    _check_ranks(A.shape, ranks)
    U = []
    for m in range(A.ndim):
        Up = np.asarray(U_prev[m], dtype=np.float64)
        if Up.shape != (A.shape[m], ranks[m]):
            raise ValueError(f"U_prev[{m}] must be a_m x r_m")
        U.append(subspace_step(A, m, Up))
    return core_tensor(A, U), U


def asi_cold_start(A: np.ndarray, Omega: list):
    """Algorithm 1 for t = 0 with explicit Gaussian test matrices."""
    A = np.asarray(A, dtype=np.float64)
    U = [cold_start_step(A, m, Omega[m]) for m in range(A.ndim)]
    return core_tensor(A, U), U


def reconstruct(S: np.ndarray, U: list) -> np.ndarray:
    """A~ = S x_1 U_1 x_2 U_2 ... x_n U_n (the Tucker form of Sec. 3.2)."""
    T = np.asarray(S, dtype=np.float64)
    for m, Um in enumerate(U):
        T = mode_product(T, np.asarray(Um, dtype=np.float64), m)
    return T


# --------------------------------------------------------------------------
# Weight gradient (Sec. 3.1 definition; appendix cost model C_ASI)
# --------------------------------------------------------------------------
def conv_out_size(H, k, stride, pad):
    return (H + 2 * pad - k) // stride + 1


def conv_wgrad_direct(A, dY, kh, kw, stride=1, pad=0, groups=1):
    """Vanilla weight gradient dW = conv(A, dY) (Sec. 3.1, first display):
      dW[c', c, i, j] = sum_{b, h', w'} dY[b, c', h', w'] * Apad[b, g(c') + c, h' s + i - p, w' s + j - p]
    with zero padding p, stride s and (for groups > 1) input channels taken
    from the group of c'.  One library contraction per kernel tap."""
    A = np.asarray(A, dtype=np.float64)
    dY = np.asarray(dY, dtype=np.float64)
    B, C, H, W = A.shape
    _, Co, Ho, Wo = dY.shape
    assert Ho == conv_out_size(H, kh, stride, pad) and Wo == conv_out_size(W, kw, stride, pad)
    assert C % groups == 0 and Co % groups == 0
    cg, og = C // groups, Co // groups
    Ap = np.zeros((B, C, H + 2 * pad, W + 2 * pad))
    Ap[:, :, pad:pad + H, pad:pad + W] = A
    dW = np.zeros((Co, cg, kh, kw))
    for g in range(groups):
        dYg = dY[:, g * og:(g + 1) * og]
        for i in range(kh):
            for j in range(kw):
                win = Ap[:, g * cg:(g + 1) * cg,
                         i:i + stride * (Ho - 1) + 1:stride,
                         j:j + stride * (Wo - 1) + 1:stride]
                dW[g * og:(g + 1) * og, :, i, j] = np.tensordot(
                    dYg, win, axes=([0, 2, 3], [0, 2, 3]))
    return dW


def conv_wgrad_factored(S, U, dY, kh, kw, stride=1, pad=0, groups=1):
    """Weight gradient from the compressed activation, in the order the five
    terms of C_ASI (appendix, "Speedup") fix:
      term 1   Z1 = dY x_1 U_1^T                      [r1, C', H', W']
      term 2-3 Z3 = S x_3 U_3 x_4 U_4                 [r1, r2, H, W]
      term 4   Z4 = conv_wgrad(Z3, Z1)                [C', r2, kh, kw]
               (pseudo-batch r1, pseudo-channels r2, same kernel/stride/pad)
      term 5   dW = Z4 x_2 U_2                        [C', C, kh, kw]
    groups == C (depthwise; the paper does not discuss it): the channel
    product pairs c' with its own row of U_2,
      dW[c, 0, i, j] = sum_k U_2[c, k] Z4[c, k, i, j].
    Other group counts: per-group rows of U_2."""
    S = np.asarray(S, dtype=np.float64)
    dY = np.asarray(dY, dtype=np.float64)
    U1, U2, U3, U4 = [np.asarray(u, dtype=np.float64) for u in U]
    C = U2.shape[0]
    Co = dY.shape[1]
    Z1 = mode_product(dY, U1.T, 0)
    Z3 = mode_product(mode_product(S, U3, 2), U4, 3)
    Z4 = conv_wgrad_direct(Z3, Z1, kh, kw, stride, pad, groups=1)   # [C', r2, kh, kw]
    if groups == 1:
        return mode_product(Z4, U2, 1)
    cg, og = C // groups, Co // groups
    dW = np.zeros((Co, cg, kh, kw))
    for g in range(groups):
        dW[g * og:(g + 1) * og] = mode_product(
            Z4[g * og:(g + 1) * og], U2[g * cg:(g + 1) * cg], 1)
    return dW


def linear_wgrad_direct(A, dY):
    """Fully-connected layer y = x W^T on token tensors: dW[o, d] =
    sum over all leading indices of dY[.., o] * A[.., d] (the paper's footnote
    in Sec. 3.1 states the conv analysis carries over; this is the standard
    definition)."""
    A = np.asarray(A, dtype=np.float64)
    dY = np.asarray(dY, dtype=np.float64)
    return dY.reshape(-1, dY.shape[-1]).T @ A.reshape(-1, A.shape[-1])


def linear_wgrad_factored(S, U, dY):
    """Same contraction order as the conv case, for an n-mode token tensor whose
    last mode is the feature mode: project dY on every leading factor, contract
    with the core over the leading ranks, expand the feature mode last."""
    S = np.asarray(S, dtype=np.float64)
    Z = np.asarray(dY, dtype=np.float64)
    nlead = S.ndim - 1
    for m in range(nlead):
        Z = mode_product(Z, np.asarray(U[m], dtype=np.float64).T, m)   # [r1,..,r_{n-1}, Dout]
    lead = list(range(nlead))
    Z4 = np.tensordot(Z, S, axes=(lead, lead))                          # [Dout, r_n]
    return Z4 @ np.asarray(U[-1], dtype=np.float64).T                   # [Dout, Din]


# --------------------------------------------------------------------------
# Closed forms (Sec. 3.2 storage; appendix overhead / speed-up / space)
# --------------------------------------------------------------------------
def compressed_elems(shape, ranks) -> int:
    """M_i = prod r_m + sum D_m r_m (Sec. 3.2, storage equation)."""
    return int(np.prod(ranks)) + int(sum(d * r for d, r in zip(shape, ranks)))


def ratio_RC(shape, ranks) -> float:
    """R_C = prod D_m / M_i (appendix, "Space complexity")."""
    return float(np.prod(shape)) / compressed_elems(shape, ranks)


def macs_O_ASI(shape, ranks) -> int:
    """O_ASI = sum_m (2 d d' r_m + r_m^3), d d' = prod D (appendix, "Overhead")."""
    n = int(np.prod(shape))
    return int(sum(2 * n * r + r ** 3 for r in ranks))


def macs_C_ASI(shape, ranks, Co, Ho, Wo, k) -> int:
    """C_ASI, five terms (appendix, "Speedup"); square k x k kernel."""
    B, C, H, W = shape
    r1, r2, r3, r4 = ranks
    return int(r1 * B * Co * Ho * Wo + r1 * r2 * r3 * r4 * H + r1 * r2 * r4 * H * W
               + r1 * r2 * Co * Ho * Wo * k * k + r2 * Co * C * k * k)


def macs_C_vanilla(shape, Co, Ho, Wo, k) -> int:
    """C_vanilla = D^2 C C' B H' W' (appendix)."""
    B, C, _, _ = shape
    return int(k * k * C * Co * B * Ho * Wo)


def macs_O_vanilla(shape, Co, k) -> int:
    """O_vanilla = D^2 C C' B H W as printed (appendix)."""
    B, C, H, W = shape
    return int(k * k * C * Co * B * H * W)


# --------------------------------------------------------------------------
# HOSVD_eps rank rule (Sec. 3.2: truncate each mode by explained variance)
# --------------------------------------------------------------------------
def mode_spectrum(A, m):
    """Eigenvalues of A_m A_m^T (squared singular values of the unfolding),
    descending."""
    Am = unfold(A, m)
    lam = np.linalg.eigvalsh(Am @ Am.T)[::-1]
    return np.maximum(lam, 0.0)


def hosvd_energy_ranks(A, eps, r_max=64):
    """Smallest r_m whose leading eigenvalues hold a fraction >= eps of the
    mode-m energy, clipped to [1, min(r_max, a_m, b_m)]."""
    A = np.asarray(A, dtype=np.float64)
    n = A.size
    ranks = []
    for m in range(A.ndim):
        lam = mode_spectrum(A, m)
        frac = np.cumsum(lam) / np.sum(lam)
        r = int(np.searchsorted(frac, eps - 1e-15) + 1)
        ranks.append(max(1, min(r, r_max, A.shape[m], n // A.shape[m])))
    return ranks


# --------------------------------------------------------------------------
# Comparison helpers used by parity tests
# --------------------------------------------------------------------------
def projector(Um):
    Um = np.asarray(Um, dtype=np.float64)
    return Um @ Um.T


def rel_fro(x, ref):
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    d = np.linalg.norm(x - ref)
    n = np.linalg.norm(ref)
    return d / n if n > 0 else d


def sign_align(S, U, U_ref):
    """Flip column j of U_m (and the matching slice of the core) by
    sign<u_{m,j}, u^{ref}_{m,j}> so two results that differ only by column
    signs compare equal."""
    S = np.array(S, dtype=np.float64, copy=True)
    U_out = []
    for m, (Um, Ur) in enumerate(zip(U, U_ref)):
        Um = np.array(Um, dtype=np.float64, copy=True)
        s = np.sign(np.sum(Um * np.asarray(Ur, dtype=np.float64), axis=0))
        s[s == 0] = 1.0
        U_out.append(Um * s[None, :])
        shape = [1] * S.ndim
        shape[m] = -1
        S = S * s.reshape(shape)
    return S, U_out
