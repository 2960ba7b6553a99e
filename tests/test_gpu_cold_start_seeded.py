"""Cold start with the library's own Gaussian test matrices (Algorithm 1, t = 0): the counter-based generator
word for word against the oracle's, the Gaussian values to fp32 rounding, and asi_init_factors_seeded against the
oracle's cold start fed with the oracle's own Omega of the same seed."""
import numpy as np
import pytest

from asi_inputs.configs import LayerSpec
from asi_inputs.generator import LayerStream
from oracle import asi_oracle as O
from oracle import gaussian_stream as gs

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _binding():
    from paper_2505_05086_b200 import binding
    return binding


@pytest.mark.parametrize("seed,stream,n_groups", [(0, 0, 1), (20250505, 3, 5000), (0xFEDCBA9876543210, 1, 777)])
def test_generator_words_are_bit_identical_to_the_oracle(seed, stream, n_groups):
    out = torch.zeros(4 * n_groups, dtype=torch.int32, device="cuda")
    _binding().philox_words(seed, stream, n_groups, out.data_ptr())
    torch.cuda.synchronize()
    got = out.cpu().numpy().view(np.uint32).reshape(n_groups, 4)
    assert np.array_equal(got, gs.words(seed, stream, n_groups))


@pytest.mark.parametrize("n,offset", [(4096, 0), (4099, 0), (1021, 1), (3, 0)])
def test_gaussian_stream_matches_the_oracle_to_fp32_rounding(n, offset):
    buf = torch.full((n + offset + 8,), 7.0, dtype=torch.float32, device="cuda")
    _binding().gaussian_stream(99, 2, n, buf.data_ptr() + 4 * offset)
    torch.cuda.synchronize()
    host = buf.cpu().numpy()
    want = gs.gaussian(99, 2, n)
    # fp32 log, sqrt, sin and cos against fp64: a few units in the last place of values up to ~6
    assert np.max(np.abs(host[offset:offset + n].astype(np.float64) - want)) < 5e-6
    assert np.all(host[:offset] == 7.0) and np.all(host[offset + n:] == 7.0)      # nothing outside [0, n)


def _seeded_case(L, A, bf16, tol, seed=4242):
    from tests.gpu_util import make_runner
    from paper_2505_05086_b200.binding import ASI_OK
    run = make_runner(L, bf16=bf16)
    run.init_factors_seeded(run.to_device(A), seed)
    assert run.plan.poll_status(run.ws_seed.data_ptr(), 0) == ASI_OK
    Omega = gs.omega_matrices(seed, L.dims, L.ranks)
    S_ref, U_ref = O.asi_cold_start(A.astype(np.float64), Omega)
    U_gpu = run.factors()
    for ug, ur in zip(U_gpu, U_ref):
        assert O.rel_fro(O.projector(ug), O.projector(ur)) < tol, L.dims
    S_al, _ = O.sign_align(run.core_np(), U_gpu, U_ref)
    assert O.rel_fro(S_al, S_ref) < tol, L.dims
    return run, [u.copy() for u in U_gpu]


def test_seeded_cold_start_generic_conv_and_its_determinism():
    dims, ranks = (5, 14, 6, 7), (2, 4, 3, 3)
    L = LayerSpec("t", "conv", dims, 4, 3, 1, 1, 1, ranks=ranks)
    A, _ = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=3).next()
    run, U1 = _seeded_case(L, A, False, 1e-4)
    run.init_factors_seeded(run.to_device(A), 4242)                  # same seed: the same bits
    for a, b in zip(U1, run.factors()):
        assert np.array_equal(a, b)
    run.init_factors_seeded(run.to_device(A), 4243)                  # another seed: another basis
    assert any(not np.array_equal(a, b) for a, b in zip(U1, run.factors()))


@pytest.mark.parametrize("dims,ranks", [((64, 512, 7, 7), (4, 4, 4, 4)), ((8, 32, 16, 16), (4, 8, 8, 8))])
def test_seeded_cold_start_on_fused_small_map_plans(dims, ranks):
    L = LayerSpec("t", "conv", dims, 8, 3, 1, 1, 1, ranks=ranks)
    A, _ = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=17).next()
    _seeded_case(L, A, False, 1e-4)


def test_seeded_cold_start_on_a_bf16_token_layer():
    dims, ranks = (4, 72, 128), (3, 16, 32)
    L = LayerSpec("t", "linear", dims, 24, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=29, rho=(0.6, 0.93, 0.96),
                     gen_ranks=(4, 32, 64), bf16=True)
    A, _ = st.next()
    _seeded_case(L, A, True, 1e-3)


def test_seeded_cold_start_rejects_a_short_workspace():
    from tests.gpu_util import make_runner
    from paper_2505_05086_b200.binding import AsiError
    dims, ranks = (5, 14, 6, 7), (2, 4, 3, 3)
    L = LayerSpec("t", "conv", dims, 4, 3, 1, 1, 1, ranks=ranks)
    run = make_runner(L)
    need = run.plan.init_seeded_ws_bytes()
    assert need > run.ws_c.numel()
    ws = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    A = torch.zeros(dims, dtype=torch.float32, device="cuda")
    with pytest.raises(AsiError):
        run.plan.init_factors_seeded(A.data_ptr(), 1, run.U[0].data_ptr(), run.core.data_ptr(), ws.data_ptr(),
                                     ws.numel())
