"""The seeded input generator: shapes, determinism, structure (low multilinear rank + small
noise, slow drift) and bf16 rounding."""
import numpy as np

from asi_inputs.configs import get_config, make_stream
from asi_inputs.generator import LayerStream, round_to_bf16, to_bf16_bits


def test_config_tables_shapes():
    c2 = get_config(1)
    assert [L.dims for L in c2.layers] == [(64, 256, 14, 14)] + [(64, 512, 7, 7)] * 3
    assert c2.layers[0].dy_shape == (64, 512, 7, 7) and c2.layers[0].dw_shape == (512, 256, 3, 3)
    c3 = get_config(2)
    assert c3.layers[2].groups == 960 and c3.layers[2].dw_shape == (960, 1, 3, 3)
    c4 = get_config(3)
    assert sum(L.count for L in c4.layers if L.k == 3) == 32
    c5 = get_config(4)
    assert c5.layers[1].dy_shape == (32, 197, 768) and c5.layers[1].dw_shape == (768, 3072)
    for idx in range(5):
        for L in get_config(idx).layers:
            n = int(np.prod(L.dims))
            assert all(1 <= r <= min(d, n // d, 64) for r, d in zip(L.ranks, L.dims))


def test_stream_is_deterministic_and_drifts_slowly():
    cfg = get_config(0)
    s1, s2 = make_stream(cfg, 0), make_stream(cfg, 0)
    A0, dY0 = s1.next()
    B0, eY0 = s2.next()
    np.testing.assert_array_equal(A0, B0)
    np.testing.assert_array_equal(dY0, eY0)
    A1, _ = s1.next()
    assert A0.dtype == np.float32 and A0.shape == (8, 32, 16, 16) and dY0.shape == (8, 32, 16, 16)
    rel = np.linalg.norm(A1 - A0) / np.linalg.norm(A0)
    assert 1e-3 < rel < 0.1
    assert abs(np.sqrt(np.mean(A0.astype(np.float64) ** 2)) - 1.0) < 1e-2
    for u, r in zip(s1.u_prev0(), cfg.layers[0].ranks):
        assert u.shape[1] == r
        np.testing.assert_allclose(u.T.astype(np.float64) @ u, np.eye(r), atol=1e-5)


def test_clip_and_bf16():
    st = LayerStream(dims=(4, 6, 5, 5), ranks=(2, 2, 2, 2), dy_shape=(4, 3, 5, 5), seed=1,
                     clip=(0.0, 6.0), bf16=True)
    A, dY = st.next()
    assert A.min() >= 0.0 and A.max() <= 6.0 and (A == 0).mean() > 0.2
    np.testing.assert_array_equal(round_to_bf16(A), A)
    assert to_bf16_bits(A).dtype == np.uint16
    back = (to_bf16_bits(dY).astype(np.uint32) << 16).view(np.float32)
    np.testing.assert_array_equal(back, dY)


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -2.5], dtype=np.float32)
    np.testing.assert_array_equal(round_to_bf16(x),
                                  np.array([1.0, 1.0, 1.0 + 2 ** -7, 1.0 + 2 ** -6, -2.5], np.float32))


def test_skip_replays_the_drift_exactly():
    from asi_inputs.generator import LayerStream
    kw = dict(dims=(4, 6, 5, 5), ranks=(2, 3, 2, 2), dy_shape=(4, 3, 5, 5), seed=77)
    a, b = LayerStream(**kw), LayerStream(**kw)
    for _ in range(5):
        a.next()
    b.skip(5)
    A1, d1 = a.next()
    A2, d2 = b.next()
    np.testing.assert_array_equal(A1, A2)
    np.testing.assert_array_equal(d1, d2)
    # the previous-step factors offered before a step span (nearly) the subspace that step will find
    c = LayerStream(**kw)
    c.skip(3)
    U = c.u_prev_now()
    assert [u.shape for u in U] == [(4, 2), (6, 3), (5, 2), (5, 2)]
    for u in U:
        assert np.allclose(u.T @ u, np.eye(u.shape[1]), atol=1e-5)
