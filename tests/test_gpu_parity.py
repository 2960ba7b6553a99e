"""CUDA path vs fp64 oracle, element by element, through the C ABI, on seeded inputs.

Tolerances (relative Frobenius error): fp32 inputs -- projectors U U^T <= 1e-4, sign-aligned
core <= 1e-4, dW <= 5e-4; bf16-input mode -- <= 2e-2 on all three."""
import numpy as np
import pytest
import torch

from asi_inputs.configs import LayerSpec, get_config, make_stream
from asi_inputs.generator import LayerStream
from oracle import asi_oracle as O
from tests.gpu_util import TOL_BF16, TOL_F32, check, compare_step, make_runner, oracle_wgrad

pytestmark = pytest.mark.gpu


def _run_config(cfg, layer_index, steps, tol, bf16=None):
    L = cfg.layers[layer_index]
    st = make_stream(cfg, layer_index)
    run = make_runner(L, bf16=cfg.bf16)
    U_prev = st.u_prev0()
    worst = {}
    for t in range(steps):
        A, dY = st.next()
        err, U_prev = compare_step(run, L, A, dY, U_prev)
        check(err, tol, f"{cfg.name}/{L.name}/step{t}")
        for k, v in err.items():
            worst[k] = max(worst.get(k, 0.0), v) if k != "sign" else min(worst.get(k, 1.0), v)
    return worst


def test_config1_single_conv_three_warm_steps():
    _run_config(get_config(0), 0, 3, TOL_F32)


def _rho(r):
    """Per-mode decay that keeps sigma_r / sigma_1 >= 0.25 whatever the rank: the one-step map has
    condition number (sigma_1 / sigma_r)^2, and fp32 accumulation times that must stay below the
    1e-4 bar."""
    return min(0.7, 0.25 ** (1.0 / max(r - 1, 1)))


SMALL = [  # ragged sizes spanning several tiles with tails; (dims, ranks, cout, k, s, p, groups)
    ((5, 12, 9, 11), (3, 5, 4, 6), 7, 3, 1, 1, 1),
    ((6, 10, 13, 13), (2, 3, 3, 3), 9, 3, 2, 1, 1),
    ((4, 16, 7, 7), (3, 4, 3, 3), 16, 3, 1, 1, 16),      # depthwise
    ((9, 24, 6, 5), (4, 6, 2, 2), 20, 1, 1, 0, 1),       # pointwise
    ((7, 8, 10, 10), (3, 3, 3, 3), 12, 1, 2, 0, 4),      # strided 1x1, four groups
    ((6, 70, 6, 6), (4, 33, 4, 4), 5, 3, 1, 1, 1),       # rank above 32 in one mode
    ((2, 3, 4, 5), (2, 3, 4, 5), 3, 3, 1, 1, 1),         # full rank everywhere
    ((1, 40, 8, 8), (1, 4, 3, 3), 6, 5, 1, 2, 1),        # batch of one, 5x5 kernel
]


@pytest.mark.parametrize("case", SMALL)
def test_small_ragged_conv_layers(case):
    dims, ranks, cout, k, s, p, g = case
    L = LayerSpec("t", "conv", dims, cout, k, s, p, g, ranks=ranks)
    rho = (0.9, 0.97, 0.9, 0.9) if max(ranks) > 8 else tuple(_rho(r) for r in ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=sum(dims) + k, rho=rho,
                     gen_ranks=tuple(min(d, max(r + 2, 4)) for d, r in zip(dims, ranks)))
    run = make_runner(L)
    U_prev = st.u_prev0()
    for t in range(2):
        A, dY = st.next()
        err, U_prev = compare_step(run, L, A, dY, U_prev)
        check(err, TOL_F32, str(case))


FUSED = [  # shapes the fused small-map kernels cover; (dims, ranks, cout, k, s, p, groups, bf16)
    ((8, 12, 7, 7), (3, 4, 3, 2), 10, 3, 1, 1, 1, False),
    ((16, 20, 7, 7), (5, 8, 4, 4), 12, 1, 1, 0, 1, False),        # ranks in the 5..8 bucket, 1x1
    ((8, 16, 7, 7), (2, 3, 3, 3), 16, 3, 1, 1, 16, False),        # depthwise
    ((16, 6, 14, 14), (4, 3, 4, 4), 8, 3, 2, 1, 1, False),        # stride 2: 14x14 -> 7x7
    ((8, 5, 14, 14), (3, 5, 6, 5), 6, 3, 1, 1, 1, False),         # 14x14 with ranks above 4
    ((8, 4, 16, 16), (2, 4, 4, 4), 4, 5, 1, 2, 1, False),         # 16x16, 5x5 kernel
    ((24, 8, 7, 7), (4, 4, 4, 4), 6, 3, 1, 1, 2, True),           # bf16 inputs, two groups
]


@pytest.mark.parametrize("case", FUSED)
def test_fused_small_map_kernels(case):
    dims, ranks, cout, k, s, p, g, bf16 = case
    L = LayerSpec("t", "conv", dims, cout, k, s, p, g, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=sum(dims) + 7 * k,
                     rho=tuple(_rho(r) for r in ranks), bf16=bf16,
                     gen_ranks=tuple(min(d, max(r + 2, 4)) for d, r in zip(dims, ranks)))
    run = make_runner(L, bf16=bf16)
    assert run.plan.launch_count(0) == 3 and run.plan.launch_count(1) == 1   # fused path chosen
    gen = make_runner(L, bf16=bf16, generic_only=True)
    assert gen.plan.launch_count(0) > 3
    U_prev = st.u_prev0()
    for t in range(2):
        A, dY = st.next()
        err_g, _ = compare_step(gen, L, A, dY, U_prev)
        check(err_g, TOL_F32, f"generic {case}")
        err, U_prev = compare_step(run, L, A, dY, U_prev)
        check(err, TOL_F32, f"fused {case}")


def test_full_rank_reproduces_vanilla_gradient():
    dims, cout = (3, 6, 5, 4), 5
    L = LayerSpec("t", "conv", dims, cout, 3, 1, 1, 1, ranks=dims)
    rng = np.random.default_rng(0)
    A = rng.standard_normal(dims).astype(np.float32)
    dY = rng.standard_normal(L.dy_shape).astype(np.float32)
    U_prev = [np.linalg.qr(rng.standard_normal((d, d)))[0].astype(np.float32) for d in dims]
    run = make_runner(L)
    run.set_factors(U_prev)
    run.compress(run.to_device(A))
    run.wgrad(run.to_device(dY))
    vanilla = O.conv_wgrad_direct(A, dY, 3, 3, 1, 1)
    assert O.rel_fro(run.dW_np(L.dw_shape), vanilla) < 5e-5
    assert O.rel_fro(O.reconstruct(run.core_np(), run.factors()), A) < 5e-5


# The modes of a Tucker tensor share one core, so a mode cannot hold more significant
# components than the other modes leave it; spectra and generating ranks below keep
# cond(A_m A_m^T U_prev) under ~100 in every mode (checked in fp64).
LINEAR = [  # (dims, ranks, cout, rho, generating ranks)
    ((6, 37, 50), (3, 5, 7), 21, (0.5, 0.67, 0.7), (6, 10, 14)),
    ((45, 33), (6, 9), 17, (0.9, 0.9), (12, 12)),
    ((8, 40, 130), (4, 16, 64), 40, (0.8, 0.95, 0.985), (8, 32, 128)),
    # batch modes of 12 / 20 / 3 rows on the register-streaming kernel (two, four and one lane per column quad;
    # the last row group of the 20-row case is idle, the 3-row case re-reads its last row; 450 quads leave a
    # ragged warp), a 100-long token mode on the cluster mode product, 128 leading indices split in two shares
    ((12, 100, 64), (5, 12, 8), 24, (0.75, 0.9, 0.85), (10, 24, 16)),
    ((20, 24, 36), (8, 16, 8), 40, (0.85, 0.93, 0.85), (16, 24, 16)),
    ((3, 50, 36), (2, 6, 6), 19, (0.5, 0.8, 0.8), (3, 12, 12)),
]


@pytest.mark.parametrize("dims,ranks,cout,rho,gen", LINEAR)
def test_linear_layers(dims, ranks, cout, rho, gen):
    L = LayerSpec("t", "linear", dims, cout, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=11 + len(dims), rho=rho,
                     gen_ranks=gen)
    run = make_runner(L)
    U_prev = st.u_prev0()
    for t in range(2):
        A, dY = st.next()
        err, U_prev = compare_step(run, L, A, dY, U_prev)
        check(err, TOL_F32, f"linear {dims}")


# bf16 token layers whose last-mode products (V_3 = A_(3)^T U_3, the first core product and, when the token
# count is a multiple of 8, the expansion P_3 = A_(3) V_3) take the tensor-core kernels: last dimension a
# multiple of 64, last rank 16 / 32 / 48 / 64, at least 128 tokens; the token counts leave ragged tiles.  With
# a token-mode rank of 16 / 32 the token-mode products V_2, P_2 run there as well (3-D TMA boxes).
LINEAR_TC = [  # (dims, ranks, cout, rho, generating ranks)
    ((4, 40, 128), (3, 6, 16), 24, (0.6, 0.8, 0.93), (4, 12, 32)),
    ((2, 197, 192), (2, 8, 32), 40, (0.5, 0.85, 0.96), (2, 16, 64)),
    ((3, 100, 320), (3, 8, 48), 32, (0.6, 0.85, 0.975), (3, 16, 96)),
    ((8, 64, 256), (4, 8, 64), 48, (0.7, 0.85, 0.985), (8, 16, 128)),
    ((4, 48, 192), (3, 6, 32), 24, (0.6, 0.8, 0.96), (4, 12, 64)),      # expansion tile with 64 valid rows
    ((4, 72, 128), (3, 16, 16), 24, (0.6, 0.93, 0.93), (4, 32, 32)),    # token mode on the tensor cores too
    ((2, 197, 192), (2, 32, 32), 40, (0.5, 0.96, 0.96), (2, 64, 64)),   # 197 tokens: ragged K chunks and row tiles
    ((4, 72, 128), (3, 20, 24), 24, (0.6, 0.94, 0.95), (4, 40, 48)),    # ranks 20 / 24: factors zero-padded to 32 columns
    ((3, 128, 256), (3, 20, 36), 32, (0.6, 0.94, 0.965), (3, 40, 72)),  # rank 36 padded to 48
    ((12, 64, 128), (5, 8, 16), 24, (0.75, 0.85, 0.93), (10, 16, 32)),    # bf16 batch mode of 12 rows: two lanes per quad
    ((24, 40, 64), (8, 8, 16), 32, (0.85, 0.85, 0.93), (16, 16, 32)),    # 24 rows: four lanes per quad, one group idle
]


@pytest.mark.parametrize("dims,ranks,cout,rho,gen", LINEAR_TC)
def test_bf16_linear_layers_on_tensor_cores(dims, ranks, cout, rho, gen):
    L = LayerSpec("t", "linear", dims, cout, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=23 + dims[2], rho=rho, gen_ranks=gen,
                     bf16=True)
    run = make_runner(L, bf16=True)
    U_prev = st.u_prev0()
    for t in range(2):
        A, dY = st.next()
        err, U_prev = compare_step(run, L, A, dY, U_prev)
        check(err, TOL_BF16, f"bf16 linear {dims}")
        # the inputs are exact in bf16 and the factor is split into three bf16 terms: fp32 accuracy on the
        # core and dW; the first step of the rank-32/48 cases is conditioned worse than the fp32
        # projector bar allows (the fp32 SIMT kernels give the same 2e-4 .. 5e-4 there)
        check(err, dict(TOL_F32, proj=1e-3), f"bf16 linear {dims} at the fp32 bar")
        assert run.ok()


def test_ranks_above_64_take_the_plain_orthogonalize_kernels():
    """Ranks 65..128 (here 96 in the feature mode and 72 in the token mode) run through the generic
    contraction kernels and the plain fp64 Cholesky-QR; spectra are kept flat enough for fp32."""
    dims, ranks = (4, 150, 200), (3, 72, 96)
    L = LayerSpec("t", "linear", dims, 24, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=61, rho=(0.6, 0.985, 0.99),
                     gen_ranks=(4, 144, 192))
    run = make_runner(L)
    U_prev = st.u_prev0()
    for t in range(2):
        A, dY = st.next()
        err, U_prev = compare_step(run, L, A, dY, U_prev)
        check(err, TOL_F32, f"ranks {ranks} step {t}")


def test_bf16_input_mode_small():
    dims, ranks = (6, 20, 9, 9), (3, 4, 3, 3)
    L = LayerSpec("t", "conv", dims, 10, 3, 1, 1, 1, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=5, bf16=True)
    run = make_runner(L, bf16=True)
    U_prev = st.u_prev0()
    A, dY = st.next()
    err, _ = compare_step(run, L, A, dY, U_prev)
    check(err, TOL_BF16, "bf16")
    # inputs are exactly representable, arithmetic is fp32: the fp32 bar holds as well
    check(err, TOL_F32, "bf16 at fp32 bar")


def test_cold_start_with_explicit_gaussian_matrices():
    dims, ranks = (5, 14, 6, 7), (2, 4, 3, 3)
    L = LayerSpec("t", "conv", dims, 4, 3, 1, 1, 1, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=3)
    A, _ = st.next()
    rng = np.random.default_rng(1)
    n = int(np.prod(dims))
    Omega = [rng.standard_normal((n // d, r)).astype(np.float32) for d, r in zip(dims, ranks)]
    run = make_runner(L)
    om = torch.from_numpy(np.concatenate([o.ravel() for o in Omega])).cuda()
    run.init_factors(run.to_device(A), om)
    assert run.ok()
    S_ref, U_ref = O.asi_cold_start(A.astype(np.float64), [o.astype(np.float64) for o in Omega])
    U_gpu = run.factors()
    for ug, ur in zip(U_gpu, U_ref):
        assert O.rel_fro(O.projector(ug), O.projector(ur)) < 1e-4
    S_al, _ = O.sign_align(run.core_np(), U_gpu, U_ref)
    assert O.rel_fro(S_al, S_ref) < 1e-4


def _cold_start_case(L, A, bf16, tol):
    rng = np.random.default_rng(1)
    n = int(np.prod(L.dims))
    Omega = [rng.standard_normal((n // d, r)).astype(np.float32) for d, r in zip(L.dims, L.ranks)]
    run = make_runner(L, bf16=bf16)
    om = torch.from_numpy(np.concatenate([o.ravel() for o in Omega])).cuda()
    run.init_factors(run.to_device(A), om)
    assert run.ok()
    S_ref, U_ref = O.asi_cold_start(A.astype(np.float64), [o.astype(np.float64) for o in Omega])
    U_gpu = run.factors()
    for ug, ur in zip(U_gpu, U_ref):
        assert O.rel_fro(O.projector(ug), O.projector(ur)) < tol, L.dims
    S_al, _ = O.sign_align(run.core_np(), U_gpu, U_ref)
    assert O.rel_fro(S_al, S_ref) < tol, L.dims


@pytest.mark.parametrize("dims,ranks", [((64, 512, 7, 7), (4, 4, 4, 4)), ((64, 256, 14, 14), (3, 3, 3, 4)),
                                        ((8, 32, 16, 16), (4, 8, 8, 8))])
def test_cold_start_on_fused_small_map_plans(dims, ranks):
    """Branch t = 0 of Algorithm 1 on plans that take the fused kernels afterwards: the expansion
    P_m = A_m Omega_m must cover every column of the unfolding whatever split count the plan uses."""
    L = LayerSpec("t", "conv", dims, 8, 3, 1, 1, 1, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=17)
    A, _ = st.next()
    assert make_runner(L).plan.launch_count(0) == 3          # the fused plan
    _cold_start_case(L, A, False, 1e-4)


def test_cold_start_on_a_bf16_token_layer():
    """Cold start through the tensor-core expansion kernels (bf16 tokens, last rank 32, token rank 16)."""
    dims, ranks = (4, 72, 128), (3, 16, 32)
    L = LayerSpec("t", "linear", dims, 24, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=29, rho=(0.6, 0.93, 0.96),
                     gen_ranks=(4, 32, 64), bf16=True)
    A, _ = st.next()
    _cold_start_case(L, A, True, 1e-3)


def test_ragged_case_at_the_benchmark_conditioning():
    """Ranks 8 with the benchmark generator's decay 0.7 per index (condition number of the one-step map
    about 150, what the single-conv configuration has), on sizes that leave ragged tiles."""
    dims, ranks = (9, 21, 11, 13), (8, 8, 8, 8)
    L = LayerSpec("t", "conv", dims, 10, 3, 1, 1, 1, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=41)      # rho = 0.7 in every mode
    run = make_runner(L)
    U_prev = st.u_prev0()
    for t in range(2):
        A, dY = st.next()
        err, U_prev = compare_step(run, L, A, dY, U_prev)
        check(err, TOL_F32, f"rho 0.7 rank 8 step {t}")


def test_expired_device_wait_is_reported_and_the_workspace_recovers():
    """The bounded waits of the kernels end in ASI_ERR_TIMEOUT instead of hanging.  With the test
    flag the producer of the bulk copy issues nothing, so every waiting CTA runs into its (1 ms)
    limit and returns; the next ordinary call on the same workspace is healthy again."""
    from paper_2505_05086_b200.binding import ASI_ERR_TIMEOUT, ASI_FLAG_TEST_EXPIRE_WAIT, Plan
    dims, ranks = (8, 12, 7, 7), (3, 4, 3, 2)
    L = LayerSpec("t", "conv", dims, 10, 3, 1, 1, 1, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=7)
    A, dY = st.next()
    run = make_runner(L)
    stalled = Plan("conv", dims, ranks, 10, 3, 1, 1, 1, flags=ASI_FLAG_TEST_EXPIRE_WAIT)
    assert stalled.info.compress_ws_bytes == run.plan.info.compress_ws_bytes
    run.set_factors(st.u_prev0())
    act = run.to_device(A)
    s = int(torch.cuda.current_stream().cuda_stream)
    stalled.compress(act.data_ptr(), run.U[run.cur].data_ptr(), run.U[1 - run.cur].data_ptr(),
                     run.core.data_ptr(), run.ws_c.data_ptr(), run.ws_c.numel(), s)
    assert stalled.poll_status(run.ws_c.data_ptr(), s) == ASI_ERR_TIMEOUT
    err, _ = compare_step(run, L, A, dY, st.u_prev0())       # same workspace, healthy plan
    check(err, TOL_F32, "after an expired wait")
    assert run.device_status() == 0


def test_rank_deficient_iterate_is_reported_not_hidden():
    dims, ranks = (4, 6, 5, 5), (2, 3, 2, 2)
    L = LayerSpec("t", "conv", dims, 4, 3, 1, 1, 1, ranks=ranks)
    rng = np.random.default_rng(2)
    A = rng.standard_normal(dims).astype(np.float32)
    U_prev = [np.linalg.qr(rng.standard_normal((d, r)))[0].astype(np.float32) for d, r in zip(dims, ranks)]
    U_prev[1][:, 2] = U_prev[1][:, 0]          # two identical columns: P_2 has rank 2 < 3
    run = make_runner(L)
    run.set_factors(U_prev)
    run.compress(run.to_device(A))
    assert run.device_status() == 6
    with pytest.raises(O.RankDeficientError):
        O.asi_compress(A.astype(np.float64), [u.astype(np.float64) for u in U_prev])
    # a healthy call on the same workspace clears the word
    U_prev[1] = np.linalg.qr(rng.standard_normal((6, 3)))[0].astype(np.float32)
    run.set_factors(U_prev)
    run.compress(run.to_device(A))
    assert run.device_status() == 0


def test_results_are_bitwise_reproducible():
    cfg = get_config(0)
    L = cfg.layers[0]
    st = make_stream(cfg, 0)
    A, dY = st.next()
    outs = []
    for _ in range(2):
        run = make_runner(L)
        run.set_factors(st.u_prev0())
        run.compress(run.to_device(A))
        run.wgrad(run.to_device(dY))
        outs.append((np.concatenate([u.ravel() for u in run.factors()]), run.core_np(), run.dW_np(L.dw_shape)))
    for a, b in zip(outs[0], outs[1]):
        np.testing.assert_array_equal(a, b)


def test_free_running_warm_start_does_not_drift_from_oracle():
    """Without teacher forcing (each side feeds on its own previous factors) the errors stay at
    the one-step level: the iteration contracts perturbations."""
    cfg = get_config(0)
    L = cfg.layers[0]
    st = make_stream(cfg, 0)
    run = make_runner(L)
    run.set_factors(st.u_prev0())
    U_ref = [u.astype(np.float64) for u in st.u_prev0()]
    for t in range(3):
        A, dY = st.next()
        run.compress(run.to_device(A))
        run.wgrad(run.to_device(dY))
        S_ref, U_ref = O.asi_compress(A.astype(np.float64), U_ref)
        dW_ref = oracle_wgrad(L, S_ref, U_ref, dY.astype(np.float64))
        for ug, ur in zip(run.factors(), U_ref):
            assert O.rel_fro(O.projector(ug), O.projector(ur)) < 3e-4
        assert O.rel_fro(run.dW_np(L.dw_shape), dW_ref) < 1e-3


def test_step_from_host_buffers_matches_device_path():
    cfg = get_config(0)
    L = cfg.layers[0]
    st = make_stream(cfg, 0)
    A, dY = st.next()
    run = make_runner(L)
    run.set_factors(st.u_prev0())
    run.compress(run.to_device(A))
    run.wgrad(run.to_device(dY))
    p = run.plan
    pin = lambda x: torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).pin_memory()
    hA, hdY = pin(A), pin(dY)
    hUp = pin(np.concatenate([u.ravel() for u in st.u_prev0()]))
    hUn = torch.empty(p.info.u_elems).pin_memory()
    hS = torch.empty(p.info.core_elems).pin_memory()
    hdW = torch.empty(p.info.dw_elems).pin_memory()
    arena = torch.empty(p.step_host_arena_bytes(), dtype=torch.uint8, device="cuda")
    s = torch.cuda.current_stream()
    p.step_host(hA.data_ptr(), hdY.data_ptr(), hUp.data_ptr(), hUn.data_ptr(), hS.data_ptr(),
                hdW.data_ptr(), arena.data_ptr(), arena.numel(), int(s.cuda_stream))
    s.synchronize()
    np.testing.assert_array_equal(hUn.numpy(), run.U[run.cur].cpu().numpy())
    np.testing.assert_array_equal(hS.numpy(), run.core.cpu().numpy())
    np.testing.assert_array_equal(hdW.numpy(), run.dW.cpu().numpy())


def test_cuda_graph_replay_matches_direct_launches():
    """bench.py replays the step as a CUDA graph with one branch per layer; the replayed kernels (incl.
    the programmatically dependent ones) must give the bits the direct launches give."""
    cfg = get_config(1)
    li = 1
    L = cfg.layers[li]
    st = make_stream(cfg, li)
    A, dY = st.next()
    run = make_runner(L)
    a, d = run.to_device(A), run.to_device(dY)
    run.set_factors(st.u_prev0())
    run.compress(a)
    run.wgrad(d)
    torch.cuda.synchronize()
    ref = (run.U[run.cur].clone(), run.core.clone(), run.dW.clone())
    # same step again from the same previous factors, captured and replayed twice
    run.cur = 1 - run.cur
    run.set_factors(st.u_prev0())
    s = torch.cuda.Stream()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        cur = torch.cuda.current_stream()
        side.wait_stream(cur)
        run.compress(a, side)
        run.wgrad(d, side)
        cur.wait_stream(side)
    for _ in range(2):
        run.core.zero_()
        run.dW.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert run.ok()
        assert torch.equal(run.U[run.cur], ref[0])
        assert torch.equal(run.core, ref[1])
        assert torch.equal(run.dW, ref[2])


def test_cuda_graph_replay_of_a_token_layer_matches_direct_launches():
    """A 3-mode linear layer runs the passes of its modes on streams of the plan's own, forked from and joined
    to the caller's stream: captured, these become parallel branches of the graph.  The replay (and a second
    direct call) must give the bits of the first direct call."""
    dims, ranks = (4, 72, 128), (3, 16, 16)
    L = LayerSpec("t", "linear", dims, 24, ranks=ranks)
    st = LayerStream(dims=dims, ranks=ranks, dy_shape=L.dy_shape, seed=151, rho=(0.6, 0.93, 0.93),
                     gen_ranks=(4, 32, 32), bf16=True)
    A, dY = st.next()
    run = make_runner(L, bf16=True)
    a, d = run.to_device(A), run.to_device(dY)
    refs = []
    for _ in range(2):
        run.set_factors(st.u_prev0())
        run.compress(a)
        run.wgrad(d)
        torch.cuda.synchronize()
        assert run.ok()
        refs.append((run.U[run.cur].clone(), run.core.clone(), run.dW.clone()))
        run.cur = 1 - run.cur
    for x, y in zip(*refs):
        assert torch.equal(x, y)
    run.set_factors(st.u_prev0())
    s = torch.cuda.Stream()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        cur = torch.cuda.current_stream()
        side.wait_stream(cur)
        run.compress(a, side)
        run.wgrad(d, side)
        cur.wait_stream(side)
    for _ in range(2):
        run.core.zero_()
        run.dW.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert run.ok()
        assert torch.equal(run.U[run.cur], refs[0][0])
        assert torch.equal(run.core, refs[0][1])
        assert torch.equal(run.dW, refs[0][2])
