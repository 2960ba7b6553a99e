"""Parity at the full sizes of the benchmark configurations (every distinct layer shape), through
the same C-ABI calls bench.py times.  The oracle handles these sizes in seconds."""
import numpy as np
import pytest

from asi_inputs.configs import get_config, make_stream
from tests.gpu_util import TOL_BF16, TOL_F32, check, compare_step, make_runner

pytestmark = pytest.mark.gpu


def _layer_steps(cfg, li, steps, tol, generic_only=False):
    L = cfg.layers[li]
    st = make_stream(cfg, li)
    run = make_runner(L, bf16=cfg.bf16, generic_only=generic_only)
    U_prev = st.u_prev0()
    for t in range(steps):
        A, dY = st.next()
        err, U_prev = compare_step(run, L, A, dY, U_prev)
        check(err, tol, f"{cfg.name}/{L.name}/step{t}: {err}")


def _first_steps_and_last(cfg, li, tol, first=3):
    """Steps 0..first-1 teacher-forced on the oracle's factors, then the last step of the configuration's
    stream: the generator is advanced without building tensors, and the step starts from the generating
    factors one drift step back (the rule step 0 follows)."""
    L = cfg.layers[li]
    st = make_stream(cfg, li)
    run = make_runner(L, bf16=cfg.bf16)
    U_prev = st.u_prev0()
    for t in range(first):
        A, dY = st.next()
        err, U_prev = compare_step(run, L, A, dY, U_prev)
        check(err, tol, f"{cfg.name}/{L.name}/step{t}: {err}")
    st.skip(cfg.steps - 1 - first)
    U_prev = st.u_prev_now()
    A, dY = st.next()
    err, _ = compare_step(run, L, A, dY, U_prev)
    check(err, tol, f"{cfg.name}/{L.name}/step{cfg.steps - 1}: {err}")


@pytest.mark.parametrize("li", range(10))
@pytest.mark.parametrize("bf16", [False, True])
def test_config4_resnet34_sweep_at_the_benchmark_ranks(li, bf16):
    """Every shape of the sweep at the 90 % ranks bench.py uses, default kernels, fp32 and bf16 inputs:
    steps 0-2 and step 19 of the 20-step stream."""
    _first_steps_and_last(get_config(3, energy=0.9, bf16=bf16), li, TOL_BF16 if bf16 else TOL_F32)


@pytest.mark.parametrize("ci,li", [(1, 0), (1, 1), (2, 0), (2, 2), (2, 4), (4, 0), (4, 1), (5, 0), (5, 2)])
def test_last_step_of_the_other_streams(ci, li):
    cfg = get_config(ci)
    _first_steps_and_last(cfg, li, TOL_BF16 if cfg.bf16 else TOL_F32, first=1)


@pytest.mark.parametrize("generic_only", [False, True])
@pytest.mark.parametrize("li", [0, 1, 2, 3])
def test_config2_resnet18_last4(li, generic_only):
    _layer_steps(get_config(1), li, 3, TOL_F32, generic_only)


@pytest.mark.parametrize("generic_only", [False, True])
@pytest.mark.parametrize("li", [0, 1, 2, 3, 4])
def test_config3_mobilenetv2_last5(li, generic_only):
    _layer_steps(get_config(2), li, 2, TOL_F32, generic_only)


@pytest.mark.parametrize("li", [6, 9])
def test_config4_small_maps_generic_kernels(li):
    _layer_steps(get_config(3, energy=0.9), li, 1, TOL_F32, generic_only=True)


@pytest.mark.parametrize("li", range(10))
@pytest.mark.parametrize("energy", [0.8, 0.95])
def test_config4_resnet34_shapes_fp32(li, energy):
    _layer_steps(get_config(3, energy=energy), li, 1, TOL_F32)


@pytest.mark.parametrize("li", [3, 6, 9])
def test_config4_resnet34_shapes_bf16(li):
    _layer_steps(get_config(3, energy=0.9, bf16=True), li, 2, TOL_BF16)


@pytest.mark.parametrize("li", [0, 1])
def test_config5_vit_mlp_bf16(li):
    _layer_steps(get_config(4), li, 2, TOL_BF16)


@pytest.mark.parametrize("li", [0, 1, 2])
def test_config6_llm_tokens_bf16(li):
    _layer_steps(get_config(5), li, 2, TOL_BF16)


def test_share_sm_plans_match_the_oracle_on_a_large_map():
    """ASI_FLAG_SHARE_SM changes only the CTA counts of the streaming kernels (and with them the number of
    partial sums): same tolerances on a 28 x 28 layer of the sweep, sampled at its first step."""
    from paper_2505_05086_b200.binding import ASI_FLAG_SHARE_SM
    from paper_2505_05086_b200.runner import LayerRunner
    cfg = get_config(3)
    li = next(i for i, L in enumerate(cfg.layers) if L.dims[2] == 28)
    L = cfg.layers[li]
    st = make_stream(cfg, li)
    U_prev = st.u_prev0()
    A, dY = st.next()
    run = LayerRunner("conv", L.dims, L.ranks, L.cout, k=L.k, stride=L.stride, pad=L.pad, groups=L.groups,
                      flags=ASI_FLAG_SHARE_SM)
    err, _ = compare_step(run, L, A, dY, U_prev)
    check(err, TOL_F32, f"share-sm {L.dims}")
    assert run.ok()
