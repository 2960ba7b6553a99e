"""Rank selection on the device (Sec. 3.2 HOSVD_eps truncation rule, Sec. 3.3 activation perplexity)
against the fp64 oracle: mode spectra, integer ranks and ||dW - dW~||_F."""
import numpy as np
import pytest
import torch

from asi_inputs.configs import get_config, make_stream
from asi_inputs.energy_ranks import ENERGY_RANKS
from oracle import asi_oracle as O
from tests.gpu_util import make_runner

pytestmark = pytest.mark.gpu


def _spectrum(run, act):
    from paper_2505_05086_b200.binding import lib
    nd = len(run.dims)
    kmax = 128
    eig = torch.zeros(nd * kmax, dtype=torch.float64, device="cuda")
    energy = torch.zeros(nd, dtype=torch.float64, device="cuda")
    ws = torch.zeros(run.plan.spectrum_ws_bytes(), dtype=torch.uint8, device="cuda")
    run.plan.mode_spectrum(act.data_ptr(), eig.data_ptr(), energy.data_ptr(), ws.data_ptr(), ws.numel(), 0)
    return eig, energy


def _ranks(run, eig, energy, eps, r_max=64):
    out = torch.zeros(len(run.dims), dtype=torch.int32, device="cuda")
    run.plan.pick_ranks(eig.data_ptr(), energy.data_ptr(), eps, r_max, out.data_ptr(), 0)
    torch.cuda.synchronize()
    return tuple(int(v) for v in out.cpu())


LAYERS = [(ci, li) for ci, n in ((1, 4), (2, 5), (3, 10)) for li in range(n)]


@pytest.mark.parametrize("ci,li", LAYERS)
def test_energy_ranks_match_the_oracle_table(ci, li):
    """Every layer of the ResNet-18, MobileNetV2 and ResNet-34 workloads: the ranks picked on the device
    from the step-0 tensor equal the ranks the oracle picked (asi_inputs/energy_ranks.py is written by
    oracle/pick_ranks.py), at every energy level the table holds."""
    cfg = get_config(ci)
    L = cfg.layers[li]
    st = make_stream(cfg, li)
    A, _ = st.next()
    run = make_runner(L)
    eig, energy = _spectrum(run, run.to_device(A))
    torch.cuda.synchronize()
    assert abs(float(energy[0].cpu()) - float(np.sum(A.astype(np.float64) ** 2))) <= 1e-9 * float(energy[0].cpu())
    for (c, l, eps), want in ENERGY_RANKS.items():
        if (c, l) == (ci, li):
            assert _ranks(run, eig, energy, eps) == tuple(want), (ci, li, eps)


@pytest.mark.parametrize("ci,li", [(1, 0), (2, 1), (2, 2), (3, 3)])
def test_mode_spectra_match_the_oracle(ci, li):
    """Eigenvalues of A_m A_m^T: the whole spectrum for modes up to 128 long (Jacobi), the leading part for
    the channel modes beyond that (subspace iteration); 1e-5 relative on everything above 1e-6 of the top."""
    cfg = get_config(ci)
    L = cfg.layers[li]
    st = make_stream(cfg, li)
    A, _ = st.next()
    run = make_runner(L)
    eig, energy = _spectrum(run, run.to_device(A))
    torch.cuda.synchronize()
    eig = eig.cpu().numpy().reshape(len(L.dims), 128)
    for m, a in enumerate(L.dims):
        lam = O.mode_spectrum(A.astype(np.float64), m)
        k = min(a, 128)
        got, want = eig[m, :k], lam[:k]
        big = want >= 1e-6 * want[0]
        if a > 128:
            big &= np.arange(k) < 64            # the block's trailing Ritz values are only lower bounds
        assert np.max(np.abs(got[big] - want[big]) / want[big]) <= 1e-5, (ci, li, m)
        assert np.all(got[:-1] >= got[1:])                      # descending
        assert abs(float(energy[m].cpu()) - lam.sum()) <= 1e-9 * lam.sum()


def test_ranks_on_a_known_spectrum_and_the_clipping_rule():
    """A tensor with mode-1 singular values 3, 2, 1, 0.5 (eigenvalues 9, 4, 1, 0.25): cumulative fractions
    0.632, 0.912, 0.982, 1 -> ranks 1, 2, 3, 4 at eps 0.6, 0.9, 0.95, 0.99; r_max clips."""
    rng = np.random.default_rng(5)
    U, _ = np.linalg.qr(rng.standard_normal((4, 4)))
    V, _ = np.linalg.qr(rng.standard_normal((120, 4)))
    A1 = (U * np.array([3.0, 2.0, 1.0, 0.5])) @ V.T            # 4 x 120
    A = A1.reshape(4, 6, 4, 5).astype(np.float32)
    from asi_inputs.configs import LayerSpec
    L = LayerSpec("t", "conv", A.shape, 3, 3, 1, 1, 1, ranks=(2, 2, 2, 2))
    run = make_runner(L)
    eig, energy = _spectrum(run, run.to_device(A))
    torch.cuda.synchronize()
    lam = eig.cpu().numpy().reshape(4, 128)[0, :4]
    assert np.allclose(lam, [9.0, 4.0, 1.0, 0.25], rtol=1e-5)
    for eps, r in ((0.6, 1), (0.9, 2), (0.95, 3), (0.99, 4)):
        assert _ranks(run, eig, energy, eps)[0] == r == O.hosvd_energy_ranks(A, eps)[0]
    assert _ranks(run, eig, energy, 0.99, r_max=2)[0] == 2
    assert _ranks(run, eig, energy, 0.999999)[1:] == tuple(O.hosvd_energy_ranks(A, 0.999999)[1:])


def test_activation_perplexity():
    """||dW - dW~||_F between the vanilla gradient and the compressed one (Sec. 3.3) equals the oracle's norm."""
    from paper_2505_05086_b200 import binding
    cfg = get_config(1)
    L = cfg.layers[1]
    st = make_stream(cfg, 1)
    A, dY = st.next()
    run = make_runner(L)
    run.set_factors(st.u_prev0())
    run.compress(run.to_device(A))
    run.wgrad(run.to_device(dY))
    dW_full = torch.from_numpy(O.conv_wgrad_direct(A.astype(np.float64), dY.astype(np.float64), L.k, L.k, L.stride,
                                                   L.pad).astype(np.float32)).cuda().reshape(-1)
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    ws = torch.zeros(binding.perplexity_ws_bytes(), dtype=torch.uint8, device="cuda")
    binding.perplexity(dW_full.data_ptr(), run.dW.data_ptr(), dW_full.numel(), out.data_ptr(), ws.data_ptr(),
                       ws.numel(), 0)
    torch.cuda.synchronize()
    want = np.linalg.norm(dW_full.cpu().numpy().astype(np.float64) - run.dW.cpu().numpy().astype(np.float64))
    assert abs(float(out.cpu()) - want) <= 1e-10 * max(want, 1.0)
    S_ref, U_ref = O.asi_compress(A.astype(np.float64), [u.astype(np.float64) for u in st.u_prev0()])
    dW_ref = O.conv_wgrad_factored(S_ref, U_ref, dY.astype(np.float64), L.k, L.k, L.stride, L.pad, L.groups)
    ref = np.linalg.norm(O.conv_wgrad_direct(A.astype(np.float64), dY.astype(np.float64), L.k, L.k, L.stride, L.pad)
                         - dW_ref)
    assert abs(float(out.cpu()) - ref) <= 1e-4 * ref
