"""Pins of the oracle's counter-based Gaussian stream (cold start, Algorithm 1 at t = 0)."""
import os

import numpy as np

from oracle import gaussian_stream as gs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    rows = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_matches_the_published_known_answer_vectors():
    rows = _kat()
    assert len(rows) == 2
    for ctr, key, want in rows:
        got = gs.philox4x32_10(np.array(ctr), np.array(key))
        assert [int(x) for x in got] == want


def test_philox_is_a_bijection_of_the_counter_on_a_small_range():
    # distinct counters under one key give distinct outputs (the round function is a permutation)
    w = gs.words(seed=12345, stream=2, n_groups=4096)
    assert len({tuple(r) for r in w.tolist()}) == 4096
    # streams and seeds separate
    assert not np.array_equal(w, gs.words(12345, 3, 4096))
    assert not np.array_equal(w, gs.words(12346, 2, 4096))


def test_counter_layout_low_word_first_and_stream_in_word_two():
    seed = 0x299F31D0A4093822                       # key words (a4093822, 299f31d0) of the third vector
    got = gs.philox4x32_10(np.array([5, 0, 7, 0]), np.array([0xA4093822, 0x299F31D0]))
    assert np.array_equal(gs.words(seed, 7, 6)[5], got)


def test_uniforms_are_exact_fp32_numbers_strictly_inside_the_unit_interval():
    x = np.array([0, 1, 511, 512, 0xFFFFFFFF], dtype=np.uint64)
    u = gs.uniform_from_word(x)
    assert u[0] == 0.5 * 2.0 ** -23 and u[2] == u[0] and u[3] == 1.5 * 2.0 ** -23
    assert u[-1] == 1.0 - 0.5 * 2.0 ** -23
    assert np.all(u.astype(np.float32).astype(np.float64) == u)


def test_box_muller_closed_forms():
    # u_b = 1/4: cos = 0, sin = 1;  u_a = exp(-1/2): radius 1;  u_a = exp(-2): radius 2
    z0, z1 = gs.box_muller(np.array([np.exp(-0.5), np.exp(-2.0)]), np.array([0.25, 0.5]))
    assert abs(z0[0]) < 1e-15 and abs(z1[0] - 1.0) < 1e-15
    assert abs(z0[1] + 2.0) < 1e-15 and abs(z1[1]) < 1e-15


def test_stream_moments_and_independence_of_neighbours():
    z = gs.gaussian(seed=20250505, stream=1, n=400000)
    assert abs(z.mean()) < 4.0 / np.sqrt(z.size)
    assert abs(z.var() - 1.0) < 4.0 * np.sqrt(2.0 / z.size)
    assert abs(np.mean(z ** 4) - 3.0) < 0.08
    for lag in (1, 2, 3, 4):
        assert abs(np.mean(z[:-lag] * z[lag:])) < 4.0 / np.sqrt(z.size)
    # a prefix of a longer draw is the shorter draw (counter-based: no hidden state)
    assert np.array_equal(z[:1001], gs.gaussian(20250505, 1, 1001))


def test_omega_matrices_have_the_cold_start_shapes():
    om = gs.omega_matrices(7, (4, 6, 5), (2, 3, 2))
    assert [o.shape for o in om] == [(30, 2), (20, 3), (24, 2)]
    assert np.array_equal(om[1].reshape(-1), gs.gaussian(7, 1, 60))
