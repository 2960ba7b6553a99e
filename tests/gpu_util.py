"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI and the fp64
oracle on the same seeded inputs and report the three figures the tolerances are stated on."""
import numpy as np

from oracle import asi_oracle as O

TOL_F32 = dict(proj=1e-4, core=1e-4, dw=5e-4)     # relative Frobenius error, fp32 inputs
TOL_BF16 = dict(proj=2e-2, core=2e-2, dw=2e-2)    # bf16-input mode
# Beside the norms: the largest element error of dW against the largest element of the reference.
# Rounding errors are spread evenly, so this ratio sits near the Frobenius figure; a misplaced or
# missing tap moves single elements by O(1) and fails it even where the norm would pass.
DW_MAX_FACTOR = 4.0


def make_runner(L, ranks=None, bf16=False, generic_only=False):
    from paper_2505_05086_b200.runner import LayerRunner
    r = tuple(ranks if ranks is not None else L.ranks)
    if L.kind == "linear":
        return LayerRunner("linear", L.dims, r, L.cout, bf16=bf16, generic_only=generic_only)
    return LayerRunner("conv", L.dims, r, L.cout, k=L.k, stride=L.stride, pad=L.pad,
                       groups=L.groups, bf16=bf16, generic_only=generic_only)


def oracle_wgrad(L, S, U, dY):
    if L.kind == "linear":
        return O.linear_wgrad_factored(S, U, dY)
    return O.conv_wgrad_factored(S, U, dY, L.k, L.k, L.stride, L.pad, L.groups)


def compare_step(run, L, A, dY, U_prev):
    """One teacher-forced step: both sides start from the same fp32 previous factors.
    Returns (errors dict, oracle factors as fp32 for the next step)."""
    run.set_factors(U_prev)
    run.compress(run.to_device(A))
    run.wgrad(run.to_device(dY))
    assert run.ok(), "device reported a rank-deficient iterate"
    U_gpu, S_gpu, dW_gpu = run.factors(), run.core_np(), run.dW_np(L.dw_shape)
    S_ref, U_ref = O.asi_compress(A.astype(np.float64), [u.astype(np.float64) for u in U_prev])
    dW_ref = oracle_wgrad(L, S_ref, U_ref, dY.astype(np.float64))
    S_al, U_al = O.sign_align(S_gpu, U_gpu, U_ref)
    err = dict(
        proj=max(O.rel_fro(O.projector(ug), O.projector(ur)) for ug, ur in zip(U_gpu, U_ref)),
        core=O.rel_fro(S_al, S_ref),
        dw=O.rel_fro(dW_gpu, dW_ref),
        dw_max=float(np.max(np.abs(dW_gpu - dW_ref)) / max(np.max(np.abs(dW_ref)), 1e-300)),
        orth=max(np.linalg.norm(ug.astype(np.float64).T @ ug - np.eye(ug.shape[1])) for ug in U_gpu),
        sign=min(float(np.min(np.sum(ug * ur, axis=0))) for ug, ur in zip(U_gpu, U_ref)),
    )
    return err, [u.astype(np.float32) for u in U_ref]


def check(err, tol, what=""):
    assert err["proj"] <= tol["proj"], (what, err)
    assert err["core"] <= tol["core"], (what, err)
    assert err["dw"] <= tol["dw"], (what, err)
    if "dw_max" in err:
        assert err["dw_max"] <= DW_MAX_FACTOR * tol["dw"], (what, err)
    assert err["orth"] <= 1e-4, (what, err)
    assert err["sign"] > 0.0, (what, err)      # same Gram-Schmidt sign convention, no flips needed
