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
