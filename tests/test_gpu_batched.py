"""asi_compress_batched / asi_wgrad_batched: the layers of one training step in one call each way.
The batched calls must give the bits that one call per layer gives, and match the fp64 oracle."""
import numpy as np
import pytest
import torch

from asi_inputs.configs import LayerSpec, get_config, make_stream
from asi_inputs.generator import LayerStream
from oracle import asi_oracle as O
from tests.gpu_util import TOL_F32, make_runner, oracle_wgrad

pytestmark = pytest.mark.gpu


def _flat(U_list):
    return np.concatenate([np.ascontiguousarray(u, dtype=np.float32).ravel() for u in U_list])


def _check_batch(specs, streams, bf16=False, oracle_layers=()):
    from paper_2505_05086_b200.runner import StepRunner
    single = [make_runner(L, bf16=bf16) for L in specs]
    batched = [make_runner(L, bf16=bf16) for L in specs]
    step = StepRunner(batched)
    U0 = [st.u_prev0() for st in streams]
    for r, b, u in zip(single, batched, U0):
        r.set_factors(u)
        b.set_factors(u)
    for t in range(2):
        inputs = [st.next() for st in streams]
        acts = [r.to_device(A) for r, (A, _) in zip(single, inputs)]
        dys = [r.to_device(dY) for r, (_, dY) in zip(single, inputs)]
        for r, a, d in zip(single, acts, dys):
            r.compress(a)
            r.wgrad(d)
        step.compress(acts)
        step.wgrad(dys)
        torch.cuda.synchronize()
        for li, (r, b) in enumerate(zip(single, batched)):
            assert b.ok()
            assert torch.equal(r.U[r.cur], b.U[b.cur]), (t, li)
            assert torch.equal(r.core, b.core), (t, li)
            assert torch.equal(r.dW, b.dW), (t, li)
        if t == 0:
            for li in oracle_layers:
                L, (A, dY) = specs[li], inputs[li]
                S_ref, U_ref = O.asi_compress(A.astype(np.float64), [u.astype(np.float64) for u in U0[li]])
                dW_ref = oracle_wgrad(L, S_ref, U_ref, dY.astype(np.float64))
                U_gpu = batched[li].factors()
                assert max(O.rel_fro(O.projector(a), O.projector(b)) for a, b in zip(U_gpu, U_ref)) <= TOL_F32["proj"]
                assert O.rel_fro(batched[li].dW_np(L.dw_shape), dW_ref) <= TOL_F32["dw"]


def test_resnet18_last4_step_in_two_calls():
    cfg = get_config(1)          # three 7x7 layers and one 14x14 layer: two kernel variants
    _check_batch(list(cfg.layers), [make_stream(cfg, li) for li in range(4)], oracle_layers=(0, 3))


def test_mobilenetv2_last5_step_in_two_calls():
    cfg = get_config(2)          # five 7x7 layers (one depthwise), one variant: 3 + 1 launches for the step
    _check_batch(list(cfg.layers), [make_stream(cfg, li) for li in range(5)], oracle_layers=(2,))


def test_mixed_batch_fused_generic_and_linear_layers():
    specs = [LayerSpec("a", "conv", (8, 12, 7, 7), 10, 3, 1, 1, 1, ranks=(3, 4, 3, 2)),
             LayerSpec("b", "conv", (5, 12, 9, 11), 7, 3, 1, 1, 1, ranks=(3, 5, 4, 6)),       # generic kernels
             LayerSpec("c", "linear", (6, 37, 50), 21, ranks=(3, 5, 7)),
             LayerSpec("d", "conv", (16, 20, 7, 7), 12, 1, 1, 0, 1, ranks=(5, 8, 4, 4)),       # the rank 5..8 variant
             LayerSpec("e", "conv", (8, 16, 7, 7), 16, 3, 1, 1, 16, ranks=(2, 3, 3, 3))]       # depthwise, same variant as a
    streams = [LayerStream(dims=L.dims, ranks=L.ranks, dy_shape=L.dy_shape, seed=90 + i,
                           rho=tuple(min(0.7, 0.25 ** (1.0 / max(r - 1, 1))) for r in L.ranks),
                           gen_ranks=tuple(min(d, max(r + 2, 4)) for d, r in zip(L.dims, L.ranks)))
               for i, L in enumerate(specs)]
    _check_batch(specs, streams, oracle_layers=(0, 1, 2, 3, 4))
