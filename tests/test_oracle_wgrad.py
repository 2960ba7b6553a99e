"""Pins for the oracle's weight gradients: scalar-loop definitions on tiny inputs, library
routines in the cases that reduce to a GEMM / autograd convolution, the two routes against
each other, and equality with the vanilla gradient at full rank."""
import numpy as np
import pytest
import torch

from oracle import asi_oracle as O


def _conv_wgrad_scalar_loops(A, dY, kh, kw, s, p, groups):
    B, C, H, W = A.shape
    _, Co, Ho, Wo = dY.shape
    cg, og = C // groups, Co // groups
    dW = np.zeros((Co, cg, kh, kw))
    for co in range(Co):
        g = co // og
        for c in range(cg):
            for i in range(kh):
                for j in range(kw):
                    acc = 0.0
                    for b in range(B):
                        for ho in range(Ho):
                            for wo in range(Wo):
                                h, w = ho * s + i - p, wo * s + j - p
                                if 0 <= h < H and 0 <= w < W:
                                    acc += dY[b, co, ho, wo] * A[b, g * cg + c, h, w]
                    dW[co, c, i, j] = acc
    return dW


GEOMS = [  # (B, C, H, W, Co, k, s, p, groups)
    (2, 3, 5, 5, 4, 3, 1, 1, 1),
    (2, 2, 6, 7, 3, 3, 2, 1, 1),
    (1, 4, 5, 4, 4, 3, 1, 1, 4),     # depthwise
    (2, 4, 4, 4, 6, 1, 1, 0, 1),     # pointwise
    (2, 4, 6, 6, 4, 1, 2, 0, 2),     # strided 1x1, two groups
    (1, 2, 7, 7, 2, 3, 2, 0, 1),     # no padding, stride 2
]


@pytest.mark.parametrize("geom", GEOMS)
def test_direct_wgrad_matches_scalar_loops_and_autograd(geom):
    B, C, H, W, Co, k, s, p, g = geom
    rng = np.random.default_rng(sum(geom))
    A = rng.standard_normal((B, C, H, W))
    Ho, Wo = O.conv_out_size(H, k, s, p), O.conv_out_size(W, k, s, p)
    dY = rng.standard_normal((B, Co, Ho, Wo))
    dW = O.conv_wgrad_direct(A, dY, k, k, s, p, g)
    np.testing.assert_allclose(dW, _conv_wgrad_scalar_loops(A, dY, k, k, s, p, g), atol=1e-12)
    # library route: autograd of a CPU convolution
    Wt = torch.zeros((Co, C // g, k, k), dtype=torch.float64, requires_grad=True)
    y = torch.nn.functional.conv2d(torch.from_numpy(A), Wt, stride=s, padding=p, groups=g)
    assert tuple(y.shape) == dY.shape
    y.backward(torch.from_numpy(dY))
    np.testing.assert_allclose(dW, Wt.grad.numpy(), atol=1e-11)


@pytest.mark.parametrize("geom", GEOMS)
def test_factored_route_equals_direct_on_reconstruction(geom):
    B, C, H, W, Co, k, s, p, g = geom
    rng = np.random.default_rng(100 + sum(geom))
    ranks = (min(B, 2), min(C, 3), 3, 2)
    S = rng.standard_normal(ranks)
    U = [np.linalg.qr(rng.standard_normal((d, r)))[0] for d, r in zip((B, C, H, W), ranks)]
    Ho, Wo = O.conv_out_size(H, k, s, p), O.conv_out_size(W, k, s, p)
    dY = rng.standard_normal((B, Co, Ho, Wo))
    direct = O.conv_wgrad_direct(O.reconstruct(S, U), dY, k, k, s, p, g)
    factored = O.conv_wgrad_factored(S, U, dY, k, k, s, p, g)
    np.testing.assert_allclose(factored, direct, atol=1e-12)


@pytest.mark.parametrize("geom", GEOMS[:4])
def test_full_rank_compressed_wgrad_equals_vanilla(geom):
    B, C, H, W, Co, k, s, p, g = geom
    rng = np.random.default_rng(200 + sum(geom))
    dims = (B, C, H, W)
    A = rng.standard_normal(dims)
    Up = [np.linalg.qr(rng.standard_normal((d, d)))[0] for d in dims]
    S, U = O.asi_compress(A, Up)
    Ho, Wo = O.conv_out_size(H, k, s, p), O.conv_out_size(W, k, s, p)
    dY = rng.standard_normal((B, Co, Ho, Wo))
    np.testing.assert_allclose(O.conv_wgrad_factored(S, U, dY, k, k, s, p, g),
                               _conv_wgrad_scalar_loops(A, dY, k, k, s, p, g), atol=1e-10)


def test_pointwise_conv_is_one_gemm():
    rng = np.random.default_rng(7)
    A = rng.standard_normal((3, 5, 4, 4))
    dY = rng.standard_normal((3, 6, 4, 4))
    ref = dY.transpose(1, 0, 2, 3).reshape(6, -1) @ A.transpose(1, 0, 2, 3).reshape(5, -1).T
    np.testing.assert_allclose(O.conv_wgrad_direct(A, dY, 1, 1)[:, :, 0, 0], ref, atol=1e-12)


def test_wgrad_is_linear_in_dY_and_in_the_core():
    rng = np.random.default_rng(8)
    dims, ranks = (2, 3, 5, 5), (2, 2, 2, 2)
    S1, S2 = rng.standard_normal(ranks), rng.standard_normal(ranks)
    U = [np.linalg.qr(rng.standard_normal((d, r)))[0] for d, r in zip(dims, ranks)]
    d1, d2 = rng.standard_normal((2, 4, 5, 5)), rng.standard_normal((2, 4, 5, 5))
    f = lambda S, d: O.conv_wgrad_factored(S, U, d, 3, 3, 1, 1)
    np.testing.assert_allclose(f(S1, 2 * d1 - 3 * d2), 2 * f(S1, d1) - 3 * f(S1, d2), atol=1e-12)
    np.testing.assert_allclose(f(S1 + S2, d1), f(S1, d1) + f(S2, d1), atol=1e-12)


@pytest.mark.parametrize("dims,dout", [((3, 4, 5), 6), ((5, 5), 3)])
def test_linear_wgrad(dims, dout):
    rng = np.random.default_rng(9)
    A = rng.standard_normal(dims)
    dY = rng.standard_normal(dims[:-1] + (dout,))
    # scalar definition
    ref = np.zeros((dout, dims[-1]))
    Af, dYf = A.reshape(-1, dims[-1]), dY.reshape(-1, dout)
    for o in range(dout):
        for d in range(dims[-1]):
            ref[o, d] = sum(dYf[t, o] * Af[t, d] for t in range(Af.shape[0]))
    np.testing.assert_allclose(O.linear_wgrad_direct(A, dY), ref, atol=1e-12)
    # factored route on a Tucker tensor; full rank reproduces the vanilla gradient
    ranks = tuple(max(1, d - 1) for d in dims)
    ranks = tuple(min(r, A.size // d) for r, d in zip(ranks, dims))
    S = rng.standard_normal(ranks)
    U = [np.linalg.qr(rng.standard_normal((d, r)))[0] for d, r in zip(dims, ranks)]
    np.testing.assert_allclose(O.linear_wgrad_factored(S, U, dY),
                               O.linear_wgrad_direct(O.reconstruct(S, U), dY), atol=1e-12)
    Sf, Uf = O.asi_compress(A, [np.linalg.qr(rng.standard_normal((d, d)))[0] for d in dims])
    np.testing.assert_allclose(O.linear_wgrad_factored(Sf, Uf, dY), ref, atol=1e-10)
