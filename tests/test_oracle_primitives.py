"""Pins for the oracle's tensor-algebra primitives: brute-force definitions on tiny tensors,
invariants, and reductions to library routines."""
import itertools

import numpy as np
import pytest

from oracle import asi_oracle as O


def _mode_product_loops(G, Bm, m):
    """The m-mode product written as its definition, one scalar at a time."""
    out_shape = list(G.shape)
    out_shape[m] = Bm.shape[0]
    R = np.zeros(out_shape)
    for idx in itertools.product(*[range(s) for s in out_shape]):
        acc = 0.0
        for p in range(G.shape[m]):
            src = list(idx)
            src[m] = p
            acc += G[tuple(src)] * Bm[idx[m], p]
        R[idx] = acc
    return R


@pytest.mark.parametrize("m", [0, 1, 2, 3])
def test_mode_product_matches_definition(m):
    rng = np.random.default_rng(m)
    G = rng.standard_normal((2, 3, 4, 5))
    Bm = rng.standard_normal((6, G.shape[m]))
    np.testing.assert_allclose(O.mode_product(G, Bm, m), _mode_product_loops(G, Bm, m), atol=1e-13)


@pytest.mark.parametrize("m", [0, 1, 2, 3])
def test_unfold_is_fiber_matrix(m):
    rng = np.random.default_rng(10 + m)
    T = rng.standard_normal((2, 3, 4, 5))
    Tm = O.unfold(T, m)
    assert Tm.shape == (T.shape[m], T.size // T.shape[m])
    # every column is a mode-m fiber of T: same multiset of fibers
    fibers = {tuple(np.round(np.moveaxis(T, m, -1)[idx], 12))
              for idx in itertools.product(*[range(s) for i, s in enumerate(T.shape) if i != m])}
    cols = {tuple(np.round(Tm[:, j], 12)) for j in range(Tm.shape[1])}
    assert fibers == cols
    # mode product == matrix product on the unfolding
    Bm = rng.standard_normal((3, T.shape[m]))
    np.testing.assert_allclose(O.unfold(O.mode_product(T, Bm, m), m), Bm @ Tm, atol=1e-13)


def test_products_on_distinct_modes_commute_and_same_mode_compose():
    rng = np.random.default_rng(3)
    G = rng.standard_normal((3, 4, 2, 5))
    B1 = rng.standard_normal((2, 4))
    B3 = rng.standard_normal((6, 5))
    a = O.mode_product(O.mode_product(G, B1, 1), B3, 3)
    b = O.mode_product(O.mode_product(G, B3, 3), B1, 1)
    np.testing.assert_allclose(a, b, atol=1e-13)
    C1 = rng.standard_normal((7, 2))
    np.testing.assert_allclose(O.mode_product(O.mode_product(G, B1, 1), C1, 1),
                               O.mode_product(G, C1 @ B1, 1), atol=1e-13)


def test_orthonormal_columns_preserve_norm():
    rng = np.random.default_rng(4)
    S = rng.standard_normal((2, 3, 2, 2))
    Q = np.linalg.qr(rng.standard_normal((9, 3)))[0]
    assert np.isclose(np.linalg.norm(O.mode_product(S, Q, 1)), np.linalg.norm(S))


def _classical_gram_schmidt(P):
    a, r = P.shape
    Q = np.zeros((a, r))
    for j in range(r):
        v = P[:, j].copy()
        for i in range(j):
            v -= (Q[:, i] @ P[:, j]) * Q[:, i]
        Q[:, j] = v / np.linalg.norm(v)
    return Q


@pytest.mark.parametrize("a,r,seed", [(5, 5, 0), (9, 4, 1), (40, 7, 2), (3, 1, 3), (64, 16, 4)])
def test_orthogonalize_is_gram_schmidt(a, r, seed):
    rng = np.random.default_rng(seed)
    P = rng.standard_normal((a, r))
    Q = O.orthogonalize(P)
    np.testing.assert_allclose(Q.T @ Q, np.eye(r), atol=1e-13)
    R = Q.T @ P
    assert np.all(np.diag(R) > 0)
    np.testing.assert_allclose(np.tril(R, -1), 0, atol=1e-12)
    np.testing.assert_allclose(Q @ R, P, atol=1e-12)
    np.testing.assert_allclose(Q, _classical_gram_schmidt(P), atol=1e-10)
    # library QR with its signs normalised the same way
    q, rr = np.linalg.qr(P)
    np.testing.assert_allclose(Q, q * np.sign(np.diag(rr))[None, :], atol=1e-12)


def test_orthogonalize_sign_cases_and_scaling():
    # first column with negative leading entry, and a column needing a sign flip
    P = np.array([[-3.0, 1.0], [4.0, 2.0], [0.0, -5.0]])
    Q = O.orthogonalize(P)
    np.testing.assert_allclose(Q[:, 0], [-0.6, 0.8, 0.0], atol=1e-14)
    assert Q[:, 1] @ P[:, 1] > 0
    np.testing.assert_allclose(O.orthogonalize(1e-20 * P), Q, atol=1e-12)
    np.testing.assert_allclose(O.orthogonalize(P * np.array([2.0, 7.0])), Q, atol=1e-13)


def test_orthogonalize_rank_deficient_raises():
    rng = np.random.default_rng(5)
    P = rng.standard_normal((10, 3))
    P[:, 2] = P[:, 0] - 2 * P[:, 1]
    with pytest.raises(O.RankDeficientError):
        O.orthogonalize(P)
    with pytest.raises(O.RankDeficientError):
        O.orthogonalize(np.zeros((4, 2)))
