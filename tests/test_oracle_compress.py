"""Pins for Algorithm 1 as the oracle states it: exactness at full rank, exact recovery of an
exactly low-rank tensor, convergence to the truncated-HOSVD subspace (library SVD used only
here), projection identities, and the cold-start branch."""
import numpy as np
import pytest

from oracle import asi_oracle as O


def _low_rank_tensor(rng, dims, ranks):
    G = rng.standard_normal(ranks)
    Us = [np.linalg.qr(rng.standard_normal((d, r)))[0] for d, r in zip(dims, ranks)]
    return O.reconstruct(G, Us), Us


def _rand_prev(rng, dims, ranks):
    return [np.linalg.qr(rng.standard_normal((d, r)))[0] for d, r in zip(dims, ranks)]


@pytest.mark.parametrize("dims", [(3, 4, 5, 2), (4, 6, 5)])
def test_full_rank_is_exact(dims):
    rng = np.random.default_rng(0)
    A = rng.standard_normal(dims)
    S, U = O.asi_compress(A, _rand_prev(rng, dims, dims))
    for Um in U:
        np.testing.assert_allclose(Um.T @ Um, np.eye(Um.shape[1]), atol=1e-12)
    np.testing.assert_allclose(O.reconstruct(S, U), A, atol=1e-11)
    assert S.shape == tuple(dims)


def test_partial_full_rank_mode_contributes_no_error():
    rng = np.random.default_rng(1)
    dims, ranks = (5, 6, 4, 3), (5, 2, 4, 3)          # only mode 2 is truncated
    A = rng.standard_normal(dims)
    S, U = O.asi_compress(A, _rand_prev(rng, dims, ranks))
    At = O.reconstruct(S, U)
    np.testing.assert_allclose(At, O.mode_product(A, O.projector(U[1]), 1), atol=1e-11)


def test_exactly_low_rank_recovered_in_one_warm_step():
    rng = np.random.default_rng(2)
    dims, ranks = (8, 9, 6, 7), (2, 3, 2, 3)
    A, Ustar = _low_rank_tensor(rng, dims, ranks)
    S, U = O.asi_compress(A, _rand_prev(rng, dims, ranks))
    for Um, Us in zip(U, Ustar):
        np.testing.assert_allclose(O.projector(Um), O.projector(Us), atol=1e-9)
    np.testing.assert_allclose(O.reconstruct(S, U), A, atol=1e-9)
    assert np.isclose(np.linalg.norm(S), np.linalg.norm(A))


def test_warm_start_from_cold_start_result_reproduces_it_on_low_rank_input():
    rng = np.random.default_rng(3)
    dims, ranks = (6, 7, 5, 4), (2, 2, 3, 2)
    A, _ = _low_rank_tensor(rng, dims, ranks)
    Omega = [rng.standard_normal((A.size // d, r)) for d, r in zip(dims, ranks)]
    S0, U0 = O.asi_cold_start(A, Omega)
    S1, U1 = O.asi_compress(A, U0)
    for a, b in zip(U0, U1):
        np.testing.assert_allclose(O.projector(a), O.projector(b), atol=1e-9)
    np.testing.assert_allclose(O.reconstruct(S0, U0), O.reconstruct(S1, U1), atol=1e-9)


def test_cold_start_is_range_finder_of_the_unfolding():
    rng = np.random.default_rng(4)
    A = rng.standard_normal((4, 5, 3))
    m, r = 1, 2
    Om = rng.standard_normal((12, r))
    U = O.cold_start_step(A, m, Om)
    # columns must span range(A_m Omega): residual of A_m Omega against span(U) is zero
    Y = O.unfold(A, m) @ Om
    np.testing.assert_allclose(U @ (U.T @ Y), Y, atol=1e-12)


@pytest.mark.parametrize("m", [0, 1, 2, 3])
def test_repeated_iteration_converges_to_dominant_left_singular_subspace(m):
    rng = np.random.default_rng(5)
    dims, r = (7, 8, 6, 5), 2
    # spectrum with a clear gap after r in mode m
    A = rng.standard_normal(dims)
    Am = O.unfold(A, m)
    u, s, vt = np.linalg.svd(Am, full_matrices=False)
    s[:r] *= 4.0
    A = np.moveaxis((u * s @ vt).reshape([dims[m]] + [d for i, d in enumerate(dims) if i != m]), 0, m)
    U = np.linalg.qr(rng.standard_normal((dims[m], r)))[0]
    gap = (s[r] / s[r - 1]) ** 2
    err = []
    for _ in range(12):
        U = O.subspace_step(A, m, U)
        err.append(np.linalg.norm(O.projector(U) - u[:, :r] @ u[:, :r].T))
    assert err[-1] < 1e-8
    # linear convergence at (sigma_{r+1}/sigma_r)^2 per step, up to a modest constant
    assert err[6] <= 50 * gap ** 6 * max(err[0], 1e-3) + 1e-12


def test_one_step_equals_power_step_on_gram_matrix():
    """P = A_m A_m^T U_prev: the step is a block power iteration on the mode Gram matrix."""
    rng = np.random.default_rng(6)
    A = rng.standard_normal((5, 4, 3, 6))
    for m in range(4):
        Up = np.linalg.qr(rng.standard_normal((A.shape[m], 2)))[0]
        # Gram matrix by the elementwise definition: G[i,j] = <slice_i, slice_j>
        G = np.array([[np.sum(np.take(A, i, axis=m) * np.take(A, j, axis=m))
                       for j in range(A.shape[m])] for i in range(A.shape[m])])
        q, rr = np.linalg.qr(G @ Up)
        np.testing.assert_allclose(O.subspace_step(A, m, Up), q * np.sign(np.diag(rr)), atol=1e-11)


def test_projection_identities():
    rng = np.random.default_rng(7)
    dims, ranks = (6, 5, 4, 7), (3, 2, 2, 4)
    A = rng.standard_normal(dims)
    S, U = O.asi_compress(A, _rand_prev(rng, dims, ranks))
    At = O.reconstruct(S, U)
    proj = A
    for m in range(4):
        proj = O.mode_product(proj, O.projector(U[m]), m)
    np.testing.assert_allclose(At, proj, atol=1e-12)
    na, nt, nr = np.linalg.norm(A) ** 2, np.linalg.norm(At) ** 2, np.linalg.norm(A - At) ** 2
    assert np.isclose(na, nt + nr)
    assert np.isclose(np.linalg.norm(S), np.linalg.norm(At))
    # core entries are inner products with rank-one basis tensors
    i, j, k, l = 1, 0, 1, 2
    basis = np.einsum("a,b,c,d->abcd", U[0][:, i], U[1][:, j], U[2][:, k], U[3][:, l])
    assert np.isclose(S[i, j, k, l], np.sum(A * basis))


def test_modes_are_independent_of_each_other():
    """Every mode unfolds the original activation, so changing one mode's previous factor
    leaves the other modes' new factors untouched."""
    rng = np.random.default_rng(8)
    dims, ranks = (5, 6, 4, 4), (2, 3, 2, 2)
    A = rng.standard_normal(dims)
    Up = _rand_prev(rng, dims, ranks)
    _, U = O.asi_compress(A, Up)
    Up2 = list(Up)
    Up2[1] = np.linalg.qr(rng.standard_normal((6, 3)))[0]
    _, U2 = O.asi_compress(A, Up2)
    for m in (0, 2, 3):
        np.testing.assert_array_equal(U[m], U2[m])
    assert np.linalg.norm(U[1] - U2[1]) > 1e-3


def test_rank_range_enforced():
    A = np.zeros((2, 3, 4, 5)) + 1.0
    with pytest.raises(ValueError):
        O.asi_compress(A, [np.eye(2, 3), np.eye(3, 1), np.eye(4, 1), np.eye(5, 1)])


def test_energy_rank_rule_on_known_spectrum():
    # diagonal-like tensor whose mode-0 singular values are known: 3, 2, 1, 0.5
    rng = np.random.default_rng(9)
    u = np.linalg.qr(rng.standard_normal((4, 4)))[0]
    v = np.linalg.qr(rng.standard_normal((30, 4)))[0]
    Am = u * np.array([3.0, 2.0, 1.0, 0.5]) @ v.T
    A = Am.reshape(4, 5, 3, 2)
    np.testing.assert_allclose(O.mode_spectrum(A, 0), [9, 4, 1, 0.25], atol=1e-10)
    tot = 14.25
    assert O.hosvd_energy_ranks(A, 9 / tot - 1e-6)[0] == 1
    assert O.hosvd_energy_ranks(A, 9 / tot + 1e-6)[0] == 2
    assert O.hosvd_energy_ranks(A, 13.5 / tot)[0] == 3
    assert O.hosvd_energy_ranks(A, 1.0)[0] == 4
