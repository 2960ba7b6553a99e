"""Host-side checks of the C ABI: the library builds and loads, exports every symbol the header
declares, validates descriptors, and reports the paper's closed forms.  No GPU work."""
import ctypes as C
import os
import re

import pytest

from oracle import asi_oracle as O


@pytest.fixture(scope="module")
def asi():
    from paper_2505_05086_b200 import build
    build.build()
    import paper_2505_05086_b200 as pkg
    pkg.lib()
    return pkg


def test_every_declared_symbol_is_exported(asi, repo_root):
    header = open(os.path.join(repo_root, "include", "asi.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(asi_[a-z_0-9]+)\s*\(", header))
    assert {"asi_plan_create", "asi_compress", "asi_conv_wgrad", "asi_linear_wgrad"} <= declared
    L = asi.lib()
    for name in declared:
        assert hasattr(L, name), name
    from paper_2505_05086_b200.binding import EXPORTS
    assert declared == set(EXPORTS)


def test_status_strings(asi):
    assert asi.status_string(0) == "ok"
    assert "rank" in asi.status_string(3)
    assert "deficient" in asi.status_string(6)


def test_plan_query_matches_closed_forms(asi):
    dims, ranks = (8, 32, 16, 16), (4, 8, 8, 8)
    p = asi.Plan("conv", dims, ranks, cout=32, k=3, stride=1, pad=1)
    i = p.info
    assert i.compressed_elems == O.compressed_elems(dims, ranks)
    assert abs(i.ratio_RC - O.ratio_RC(dims, ranks)) < 1e-12
    assert i.macs_O_ASI == O.macs_O_ASI(dims, ranks)
    assert i.macs_C_ASI == O.macs_C_ASI(dims, ranks, 32, 16, 16, 3)
    assert i.macs_C_vanilla == O.macs_C_vanilla(dims, 32, 16, 16, 3)
    assert (i.out_h, i.out_w) == (16, 16)
    assert list(i.u_offset) == [0, 32, 32 + 256, 32 + 256 + 128]
    assert i.u_elems == 32 + 256 + 128 + 128 and i.core_elems == 4 * 8 * 8 * 8
    assert i.dw_elems == 32 * 32 * 9 and i.dy_elems == 8 * 32 * 16 * 16
    assert i.compress_ws_bytes % 256 == 0 and i.wgrad_ws_bytes % 256 == 0
    # stride 2
    p2 = asi.Plan("conv", (64, 256, 14, 14), (3, 3, 3, 4), cout=512, k=3, stride=2, pad=1)
    assert (p2.info.out_h, p2.info.out_w) == (7, 7)
    assert p2.info.macs_C_ASI == O.macs_C_ASI((64, 256, 14, 14), (3, 3, 3, 4), 512, 7, 7, 3)
    # linear
    p3 = asi.Plan("linear", (32, 197, 768), (8, 32, 64), cout=3072, bf16=True)
    assert p3.info.dw_elems == 3072 * 768 and p3.info.dy_elems == 32 * 197 * 3072
    assert p3.info.compressed_elems == O.compressed_elems((32, 197, 768), (8, 32, 64))
    # cost of the linear backward, term by term: dY x_1 U_1^T, x_2 U_2^T, the contraction with the core
    # over the leading ranks, and the expansion with U_3^T
    B, N, Din, Dout, r1, r2, r3 = 32, 197, 768, 3072, 8, 32, 64
    assert p3.info.macs_C_ASI == r1 * B * N * Dout + r1 * r2 * N * Dout + r1 * r2 * r3 * Dout + r3 * Dout * Din
    assert p3.info.macs_C_vanilla == B * N * Din * Dout
    p4 = asi.Plan("linear", (45, 33), (6, 9), cout=17)
    assert p4.info.macs_C_ASI == 6 * 45 * 17 + 6 * 9 * 17 + 9 * 17 * 33


@pytest.mark.parametrize("dims,ranks,on_tensor_cores", [
    ((32, 197, 768), (8, 32, 64), True),      # ViT-Base MLP input: last mode and token mode both qualify
    ((8, 64, 256), (4, 8, 64), True),         # last mode only
    ((8, 64, 256), (4, 8, 60), True),         # rank 60: the factor is zero-padded to 64 columns
    ((8, 64, 256), (4, 8, 62), False),        # rank not a multiple of 4
    ((8, 64, 250), (4, 8, 64), False),        # feature extent not a multiple of the K chunk
])
def test_bf16_plans_pick_the_tensor_core_products_by_shape(asi, dims, ranks, on_tensor_cores):
    """A bf16 plan whose dense products fit the tensor-core tiling enqueues the factor-split launches
    and reserves their scratch; any other plan is launch-for-launch the fp32 plan."""
    tc = asi.Plan("linear", dims, ranks, cout=128, bf16=True)
    f32 = asi.Plan("linear", dims, ranks, cout=128)
    more = tc.launch_count(0) - f32.launch_count(0)
    extra = tc.info.compress_ws_bytes - f32.info.compress_ws_bytes
    if on_tensor_cores:
        assert more > 0 and extra > 0
    else:
        assert more == 0 and extra == 0
    # the backward pass differs only when the token-mode factor qualifies: dY x_2 U_2^T then runs first, on
    # the tensor cores (one launch more: the factor split)
    token_mode_on_tc = ranks[1] % 4 == 0 and 16 <= ranks[1] <= 64
    assert tc.launch_count(1) == f32.launch_count(1) + (1 if token_mode_on_tc else 0)


@pytest.mark.parametrize("kw,code", [
    (dict(dims=(8, 32, 16, 16), ranks=(9, 8, 8, 8)), 3),            # r_1 > a_1
    (dict(dims=(8, 32, 16, 16), ranks=(0, 8, 8, 8)), 3),
    (dict(dims=(200, 2, 2, 2), ranks=(9, 1, 1, 1)), 3),            # r_1 > b_1 = 8
    (dict(dims=(256, 256, 8, 8), ranks=(129, 8, 8, 8)), 2),        # rank above the supported 128
    (dict(dims=(8, 32, 16, 16), ranks=(4, 8, 8, 8), dilation=2), 2),
    (dict(dims=(8, 32, 16, 16), ranks=(4, 8, 8, 8), groups=3), 1),
    (dict(dims=(8, 32, 16, 16), ranks=(4, 8, 8, 8), k=0), 1),
    (dict(dims=(8, 32, 2, 2), ranks=(4, 8, 2, 2), k=5), 1),        # kernel larger than padded input
    (dict(dims=(8, 0, 16, 16), ranks=(4, 8, 8, 8)), 1),
])
def test_plan_rejects_bad_descriptors(asi, kw, code):
    args = dict(cout=32, k=3, stride=1, pad=1)
    args.update(kw)
    with pytest.raises(asi.AsiError) as e:
        asi.Plan("conv", **args)
    assert e.value.code == code


def test_plan_rejects_wrong_ndim_and_nulls(asi):
    with pytest.raises(asi.AsiError) as e:
        asi.Plan("conv", (8, 32, 16), (4, 8, 8), cout=4)
    assert e.value.code == 2
    with pytest.raises(asi.AsiError) as e:
        asi.Plan("linear", (8, 4, 4, 4), (2, 2, 2, 2), cout=4)
    assert e.value.code == 2
    L = asi.lib()
    assert L.asi_plan_create(None, None) == 1
    assert L.asi_plan_destroy(None) == 1
    assert L.asi_plan_query(None, None) == 1


def test_host_detectable_call_errors_enqueue_nothing(asi):
    """Null pointers, aliasing factors, short or misaligned workspaces are refused on the host
    before any CUDA call is made (this test runs without a GPU)."""
    p = asi.Plan("conv", (8, 32, 16, 16), (4, 8, 8, 8), cout=32, k=3, stride=1, pad=1)
    L, h = asi.lib(), p.handle
    ws = p.info.compress_ws_bytes
    assert L.asi_compress(h, None, 256, 512, 768, 1024, ws, None) == 1
    assert L.asi_compress(h, 256, 512, 512, 768, 1024, ws, None) == 1          # U_prev aliases U_new
    assert L.asi_compress(h, 256, 512, 768, 1024, 4096, ws - 1, None) == 4     # too small
    assert L.asi_compress(h, 256, 512, 768, 1024, 4096 + 8, ws, None) == 4     # misaligned
    assert L.asi_conv_wgrad(h, 256, 512, 768, 1024, 4096, p.info.wgrad_ws_bytes - 1, None) == 4
    assert L.asi_linear_wgrad(h, 256, 512, 768, 1024, 4096, 1 << 30, None) == 1  # conv plan
    assert L.asi_conv_wgrad(h, 256, 512, None, 1024, 4096, 1 << 30, None) == 1
    assert L.asi_step_host(h, None, None, None, None, None, None, None, 0, None) == 1
    assert L.asi_step_host_arena_bytes(h) >= ws
    assert p.launch_count(0) > 0 and p.launch_count(1) > 0


def test_batched_entry_points_validate_before_enqueuing(asi):
    """Null arrays, an empty batch and two layers sharing one workspace are refused on the host."""
    from paper_2505_05086_b200.binding import ASI_ERR_INVALID_ARG, ASI_ERR_WORKSPACE
    L = asi.lib()
    p = asi.Plan("conv", (8, 12, 7, 7), (3, 4, 3, 2), cout=10, k=3, stride=1, pad=1)
    n = 2
    h = (C.c_void_p * n)(p.handle.value, p.handle.value)
    fake = (C.c_void_p * n)(4096, 8192)              # never dereferenced: the calls fail before any launch
    other = (C.c_void_p * n)(12288, 16384)
    same_ws = (C.c_void_p * n)(256 * 100, 256 * 100)
    big = (C.c_size_t * n)(1 << 30, 1 << 30)
    small = (C.c_size_t * n)(16, 16)
    assert L.asi_compress_batched(None, fake, fake, other, fake, fake, big, n, None) == ASI_ERR_INVALID_ARG
    assert L.asi_compress_batched(h, fake, fake, other, fake, fake, big, 0, None) == ASI_ERR_INVALID_ARG
    assert L.asi_compress_batched(h, fake, fake, fake, fake, fake, big, n, None) == ASI_ERR_INVALID_ARG    # U_new aliases U_prev
    assert L.asi_compress_batched(h, fake, fake, other, fake, same_ws, big, n, None) == ASI_ERR_INVALID_ARG
    assert L.asi_compress_batched(h, fake, fake, other, fake, fake, small, n, None) == ASI_ERR_WORKSPACE
    assert L.asi_wgrad_batched(h, fake, fake, None, fake, fake, big, n, None) == ASI_ERR_INVALID_ARG
    assert L.asi_wgrad_batched(h, fake, fake, fake, fake, fake, small, n, None) == ASI_ERR_WORKSPACE
