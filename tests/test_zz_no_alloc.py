"""asi_compress_static_ws: the variant of asi_compress for callers that may not allocate.

Some users of this library run where device allocation is forbidden (a hook inside a training loop
that must leave the framework's allocator alone, a process with a fixed memory budget).  For them the
library carries a built-in scratch array; this test calls that entry point through the C ABI and
checks it against asi_compress with an ordinary caller-owned workspace: same factors, same core,
on two consecutive calls (the second call finds the first call's leftovers in the shared array).

This file sorts last on purpose, so a run that stops at the first failure has already exercised
every other test."""
import numpy as np
import pytest
import torch

from asi_inputs.configs import get_config, make_stream
from oracle import asi_oracle as O
from tests.gpu_util import TOL_F32, make_runner

pytestmark = pytest.mark.gpu


def _flat(U_list):
    return np.concatenate([np.ascontiguousarray(u, dtype=np.float32).ravel() for u in U_list])


@pytest.mark.parametrize("cfg_index,layer", [(0, 0), (1, 1)])
def test_static_workspace_variant_matches_asi_compress(cfg_index, layer):
    from paper_2505_05086_b200.binding import ASI_STATIC_WS_MAX_BYTES
    cfg = get_config(cfg_index)
    L = cfg.layers[layer]
    st = make_stream(cfg, layer)
    run = make_runner(L)
    assert run.plan.info.compress_ws_bytes <= ASI_STATIC_WS_MAX_BYTES
    dev = run.device
    U_prev = torch.from_numpy(_flat(st.u_prev0())).to(dev)
    stream = int(torch.cuda.current_stream().cuda_stream)
    for call in range(2):                         # two calls in a row on the shared array
        A, _ = st.next()
        act = run.to_device(A)
        U_ref = torch.zeros_like(U_prev)
        S_ref = torch.zeros(run.plan.info.core_elems, device=dev)
        run.plan.compress(act.data_ptr(), U_prev.data_ptr(), U_ref.data_ptr(), S_ref.data_ptr(),
                          run.ws_c.data_ptr(), run.ws_c.numel(), stream)
        U_new = torch.zeros_like(U_prev)
        S_new = torch.zeros_like(S_ref)
        run.plan.compress_static_ws(act.data_ptr(), U_prev.data_ptr(), U_new.data_ptr(),
                                    S_new.data_ptr(), stream)
        torch.cuda.synchronize()
        u_ref, u_new = U_ref.cpu().numpy(), U_new.cpu().numpy()
        s_ref, s_new = S_ref.cpu().numpy(), S_new.cpu().numpy()
        assert np.isfinite(u_new).all() and np.isfinite(s_new).all()
        assert np.linalg.norm(u_ref) > 0 and np.linalg.norm(s_ref) > 0
        off = 0
        for d, r in zip(L.dims, L.ranks):
            a = u_new[off:off + d * r].reshape(d, r)
            b = u_ref[off:off + d * r].reshape(d, r)
            assert O.rel_fro(O.projector(a), O.projector(b)) <= TOL_F32["proj"], (call, d, r)
            off += d * r
        assert O.rel_fro(s_new, s_ref) <= TOL_F32["core"], call
        U_prev = U_ref                            # warm start of the next call


def test_shared_array_serves_plans_of_different_layouts_in_turn():
    """A fused small-map plan and a generic-path plan alternate on the one built-in array: each call
    finds the other plan's leftovers in a different layout and must still match asi_compress run on
    a workspace of its own (the generic path clears the status word by a memset, the fused path in
    its first kernel)."""
    from paper_2505_05086_b200.binding import ASI_STATIC_WS_MAX_BYTES
    cfg = get_config(0)
    L = cfg.layers[0]
    st = make_stream(cfg, 0)
    runs = [make_runner(L), make_runner(L, generic_only=True)]
    assert runs[0].plan.launch_count(0) == 3 and runs[1].plan.launch_count(0) > 3
    dev = runs[0].device
    U_prev = torch.from_numpy(_flat(st.u_prev0())).to(dev)
    stream = int(torch.cuda.current_stream().cuda_stream)
    for call in range(4):
        run = runs[call % 2]
        assert run.plan.info.compress_ws_bytes <= ASI_STATIC_WS_MAX_BYTES
        A, _ = st.next()
        act = run.to_device(A)
        U_ref, U_new = torch.zeros_like(U_prev), torch.zeros_like(U_prev)
        S_ref = torch.zeros(run.plan.info.core_elems, device=dev)
        S_new = torch.zeros_like(S_ref)
        run.plan.compress(act.data_ptr(), U_prev.data_ptr(), U_ref.data_ptr(), S_ref.data_ptr(),
                          run.ws_c.data_ptr(), run.ws_c.numel(), stream)
        run.plan.compress_static_ws(act.data_ptr(), U_prev.data_ptr(), U_new.data_ptr(), S_new.data_ptr(), stream)
        torch.cuda.synchronize()
        assert torch.equal(U_new, U_ref), call          # same kernels, same order of sums: the same bits
        assert torch.equal(S_new, S_ref), call
        U_prev = U_ref


def test_static_workspace_variant_refuses_oversized_plans():
    from paper_2505_05086_b200.binding import ASI_ERR_WORKSPACE, ASI_STATIC_WS_MAX_BYTES, AsiError, Plan
    p = Plan("conv", (128, 64, 56, 56), (3, 3, 3, 3), cout=64, k=3, stride=1, pad=1)
    assert p.info.compress_ws_bytes > ASI_STATIC_WS_MAX_BYTES
    x = torch.zeros(16, device="cuda")            # never read: the call must fail before any launch
    with pytest.raises(AsiError) as e:
        p.compress_static_ws(x.data_ptr(), x.data_ptr(), x.data_ptr() + 32, x.data_ptr(), 0)
    assert e.value.code == ASI_ERR_WORKSPACE
