"""ctypes binding of the ASI C ABI (include/asi.h).

Argument marshalling only: every step of the path runs inside the CUDA library.  Tensors are
passed as raw device pointers (``tensor.data_ptr()``); PyTorch is used by callers for device
memory and streams.  There is no CPU fallback: if the shared library is missing the import of
``lib()`` raises.
"""
from __future__ import annotations

import ctypes as C
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libasi_b200.so")
_lib = None

ASI_OK = 0
ASI_ERR_INVALID_ARG = 1
ASI_ERR_UNSUPPORTED = 2
ASI_ERR_RANK_RANGE = 3
ASI_ERR_WORKSPACE = 4
ASI_ERR_CUDA = 5
ASI_ERR_RANK_DEFICIENT = 6
ASI_ERR_TIMEOUT = 7
ASI_F32, ASI_BF16 = 0, 1
ASI_CONV2D, ASI_LINEAR = 0, 1
ASI_MAX_MODES = 4
ASI_STATIC_WS_MAX_BYTES = 4 << 20
ASI_FLAG_GENERIC_ONLY, ASI_FLAG_TEST_EXPIRE_WAIT, ASI_FLAG_SHARE_SM = 1, 2, 4

EXPORTS = (
    "asi_plan_create", "asi_plan_destroy", "asi_plan_query", "asi_compress", "asi_compress_static_ws",
    "asi_init_factors", "asi_init_seeded_ws_bytes", "asi_init_factors_seeded", "asi_gaussian_stream",
    "asi_philox_words", "asi_compress_batched", "asi_wgrad_batched",
    "asi_spectrum_ws_bytes", "asi_mode_spectrum", "asi_pick_ranks", "asi_perplexity_ws_bytes", "asi_perplexity",
    "asi_conv_wgrad", "asi_linear_wgrad", "asi_step_host_arena_bytes", "asi_step_host", "asi_step_host_status",
    "asi_poll_status", "asi_launch_count", "asi_status_string", "asi_profile_begin",
    "asi_profile_end", "asi_last_cuda_error",
)


class LayerDesc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("in_dtype", C.c_int32), ("ndim", C.c_int32),
                ("dims", C.c_int64 * ASI_MAX_MODES), ("ranks", C.c_int32 * ASI_MAX_MODES),
                ("cout", C.c_int32), ("kh", C.c_int32), ("kw", C.c_int32),
                ("stride_h", C.c_int32), ("stride_w", C.c_int32), ("pad_h", C.c_int32),
                ("pad_w", C.c_int32), ("dil_h", C.c_int32), ("dil_w", C.c_int32),
                ("groups", C.c_int32), ("flags", C.c_int32)]


class PlanInfo(C.Structure):
    _fields_ = [("compress_ws_bytes", C.c_size_t), ("wgrad_ws_bytes", C.c_size_t),
                ("u_offset", C.c_int64 * ASI_MAX_MODES), ("u_elems", C.c_int64),
                ("core_elems", C.c_int64), ("act_elems", C.c_int64), ("dy_elems", C.c_int64),
                ("dw_elems", C.c_int64), ("out_h", C.c_int64), ("out_w", C.c_int64),
                ("compressed_elems", C.c_int64), ("ratio_RC", C.c_double),
                ("macs_O_ASI", C.c_double), ("macs_C_ASI", C.c_double),
                ("macs_C_vanilla", C.c_double)]


class AsiError(RuntimeError):
    def __init__(self, code, where):
        self.code = int(code)
        detail = ""
        if self.code == ASI_ERR_CUDA:
            detail = " [" + lib().asi_last_cuda_error().decode() + "]"
        super().__init__(f"{where}: {status_string(code)} (status {int(code)}){detail}")


def lib():
    """Loads libasi_b200.so (built in-tree by paper_2505_05086_b200.build).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} not built: run `python -m paper_2505_05086_b200.build`")
    L = C.CDLL(_LIB_PATH)
    vp, sz, i32 = C.c_void_p, C.c_size_t, C.c_int32
    L.asi_plan_create.argtypes = [C.POINTER(LayerDesc), C.POINTER(vp)]
    L.asi_plan_destroy.argtypes = [vp]
    L.asi_plan_query.argtypes = [vp, C.POINTER(PlanInfo)]
    L.asi_compress.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
    L.asi_compress_static_ws.argtypes = [vp, vp, vp, vp, vp, vp]
    L.asi_init_factors.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
    L.asi_init_seeded_ws_bytes.argtypes = [vp]
    L.asi_init_seeded_ws_bytes.restype = sz
    L.asi_init_factors_seeded.argtypes = [vp, vp, C.c_uint64, vp, vp, vp, sz, vp]
    L.asi_gaussian_stream.argtypes = [C.c_uint64, C.c_uint32, C.c_int64, vp, vp]
    L.asi_philox_words.argtypes = [C.c_uint64, C.c_uint32, C.c_int64, vp, vp]
    pvp, psz = C.POINTER(vp), C.POINTER(sz)
    L.asi_compress_batched.argtypes = [pvp, pvp, pvp, pvp, pvp, pvp, psz, i32, vp]
    L.asi_wgrad_batched.argtypes = [pvp, pvp, pvp, pvp, pvp, pvp, psz, i32, vp]
    L.asi_conv_wgrad.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
    L.asi_linear_wgrad.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
    L.asi_spectrum_ws_bytes.argtypes = [vp]
    L.asi_spectrum_ws_bytes.restype = sz
    L.asi_mode_spectrum.argtypes = [vp, vp, vp, vp, vp, sz, vp]
    L.asi_pick_ranks.argtypes = [vp, vp, vp, C.c_double, i32, vp, vp]
    L.asi_perplexity_ws_bytes.argtypes = []
    L.asi_perplexity_ws_bytes.restype = sz
    L.asi_perplexity.argtypes = [vp, vp, C.c_int64, vp, vp, sz, vp]
    L.asi_step_host_arena_bytes.argtypes = [vp]
    L.asi_step_host_arena_bytes.restype = sz
    L.asi_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.asi_poll_status.argtypes = [vp, vp, vp, C.POINTER(i32)]
    L.asi_step_host_status.argtypes = [vp, vp, vp, C.POINTER(i32)]
    L.asi_launch_count.argtypes = [vp, i32]
    L.asi_launch_count.restype = i32
    L.asi_profile_begin.argtypes = [i32, C.POINTER(vp), i32]
    L.asi_profile_begin.restype = i32
    L.asi_profile_end.argtypes = [C.POINTER(C.c_double)]
    L.asi_profile_end.restype = i32
    L.asi_last_cuda_error.argtypes = []
    L.asi_last_cuda_error.restype = C.c_char_p
    L.asi_status_string.argtypes = [i32]
    L.asi_status_string.restype = C.c_char_p
    for name in ("asi_plan_create", "asi_plan_destroy", "asi_plan_query", "asi_compress", "asi_compress_static_ws",
                 "asi_init_factors", "asi_init_factors_seeded", "asi_gaussian_stream", "asi_philox_words",
                 "asi_conv_wgrad", "asi_linear_wgrad", "asi_step_host",
                 "asi_poll_status", "asi_step_host_status", "asi_compress_batched", "asi_wgrad_batched",
                 "asi_mode_spectrum", "asi_pick_ranks", "asi_perplexity"):
        getattr(L, name).restype = i32
    _lib = L
    return L


def status_string(code) -> str:
    return lib().asi_status_string(int(code)).decode()


def _check(code, where):
    if code != ASI_OK:
        raise AsiError(code, where)


def make_desc(kind, dims, ranks, cout, k=1, stride=1, pad=0, groups=1, bf16=False, dilation=1,
              generic_only=False, flags=0):
    d = LayerDesc()
    d.kind = ASI_CONV2D if kind == "conv" else ASI_LINEAR
    d.in_dtype = ASI_BF16 if bf16 else ASI_F32
    d.ndim = len(dims)
    for i, v in enumerate(dims):
        d.dims[i] = int(v)
    for i, v in enumerate(ranks):
        d.ranks[i] = int(v)
    d.cout = int(cout)
    kh, kw = (k, k) if isinstance(k, int) else k
    sh, sw = (stride, stride) if isinstance(stride, int) else stride
    ph, pw = (pad, pad) if isinstance(pad, int) else pad
    d.kh, d.kw, d.stride_h, d.stride_w, d.pad_h, d.pad_w = kh, kw, sh, sw, ph, pw
    d.dil_h = d.dil_w = int(dilation)
    d.groups = int(groups)
    d.flags = (1 if generic_only else 0) | int(flags)
    return d


class Plan:
    """Owns one asi_plan_t.  Methods mirror the C entry points one to one; pointer arguments are
    integers (device or host addresses), ``stream`` is a CUDA stream handle (0 = default)."""

    def __init__(self, kind, dims, ranks, cout, k=1, stride=1, pad=0, groups=1, bf16=False,
                 dilation=1, generic_only=False, flags=0):
        self._h = C.c_void_p()
        self.desc = make_desc(kind, dims, ranks, cout, k, stride, pad, groups, bf16, dilation,
                              generic_only, flags)
        _check(lib().asi_plan_create(C.byref(self.desc), C.byref(self._h)), "asi_plan_create")
        self.kind = kind
        self.info = PlanInfo()
        _check(lib().asi_plan_query(self._h, C.byref(self.info)), "asi_plan_query")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().asi_plan_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self):
        return self._h

    def launch_count(self, which):
        return lib().asi_launch_count(self._h, which)

    def compress(self, act, U_prev, U_new, core, ws, ws_bytes, stream=0):
        _check(lib().asi_compress(self._h, act, U_prev, U_new, core, ws, ws_bytes, stream),
               "asi_compress")

    def compress_static_ws(self, act, U_prev, U_new, core, stream=0):
        """asi_compress with the library's built-in scratch array (no workspace argument)."""
        _check(lib().asi_compress_static_ws(self._h, act, U_prev, U_new, core, stream),
               "asi_compress_static_ws")

    def init_factors(self, act, omega, U_new, core, ws, ws_bytes, stream=0):
        _check(lib().asi_init_factors(self._h, act, omega, U_new, core, ws, ws_bytes, stream),
               "asi_init_factors")

    def init_seeded_ws_bytes(self):
        return lib().asi_init_seeded_ws_bytes(self._h)

    def init_factors_seeded(self, act, seed, U_new, core, ws, ws_bytes, stream=0):
        _check(lib().asi_init_factors_seeded(self._h, act, int(seed), U_new, core, ws, ws_bytes, stream),
               "asi_init_factors_seeded")

    def conv_wgrad(self, core, U, dY, dW, ws, ws_bytes, stream=0):
        _check(lib().asi_conv_wgrad(self._h, core, U, dY, dW, ws, ws_bytes, stream), "asi_conv_wgrad")

    def linear_wgrad(self, core, U, dY, dW, ws, ws_bytes, stream=0):
        _check(lib().asi_linear_wgrad(self._h, core, U, dY, dW, ws, ws_bytes, stream),
               "asi_linear_wgrad")

    def wgrad(self, core, U, dY, dW, ws, ws_bytes, stream=0):
        if self.kind == "conv":
            self.conv_wgrad(core, U, dY, dW, ws, ws_bytes, stream)
        else:
            self.linear_wgrad(core, U, dY, dW, ws, ws_bytes, stream)

    def spectrum_ws_bytes(self):
        return lib().asi_spectrum_ws_bytes(self._h)

    def mode_spectrum(self, act, eig, energy, ws, ws_bytes, stream=0):
        _check(lib().asi_mode_spectrum(self._h, act, eig, energy, ws, ws_bytes, stream), "asi_mode_spectrum")

    def pick_ranks(self, eig, energy, eps, r_max, ranks, stream=0):
        _check(lib().asi_pick_ranks(self._h, eig, energy, float(eps), int(r_max), ranks, stream), "asi_pick_ranks")

    def step_host_arena_bytes(self):
        return lib().asi_step_host_arena_bytes(self._h)

    def step_host(self, act_h, dY_h, U_prev_h, U_new_h, core_h, dW_h, arena, arena_bytes, stream=0):
        _check(lib().asi_step_host(self._h, act_h, dY_h, U_prev_h, U_new_h, core_h, dW_h, arena,
                                   arena_bytes, stream), "asi_step_host")

    def step_host_status(self, arena, stream=0):
        out = C.c_int32(0)
        _check(lib().asi_step_host_status(self._h, arena, stream, C.byref(out)), "asi_step_host_status")
        return out.value

    def poll_status(self, ws, stream=0):
        out = C.c_int32(0)
        _check(lib().asi_poll_status(self._h, ws, stream, C.byref(out)), "asi_poll_status")
        return out.value


class Batch:
    """Argument arrays of asi_compress_batched / asi_wgrad_batched for a fixed list of plans.  The
    arrays are built once (marshalling only) and can be re-used every step with new pointers."""

    def __init__(self, plans):
        self.plans = list(plans)
        self.n = len(self.plans)
        self._h = (C.c_void_p * self.n)(*[p.handle.value for p in self.plans])

    def _arr(self, values):
        return (C.c_void_p * self.n)(*[int(v) for v in values])

    def compress(self, acts, U_prev, U_new, cores, ws, ws_bytes, stream=0):
        sizes = (C.c_size_t * self.n)(*[int(v) for v in ws_bytes])
        _check(lib().asi_compress_batched(self._h, self._arr(acts), self._arr(U_prev), self._arr(U_new),
                                          self._arr(cores), self._arr(ws), sizes, self.n, stream),
               "asi_compress_batched")

    def wgrad(self, cores, U, dY, dW, ws, ws_bytes, stream=0):
        sizes = (C.c_size_t * self.n)(*[int(v) for v in ws_bytes])
        _check(lib().asi_wgrad_batched(self._h, self._arr(cores), self._arr(U), self._arr(dY), self._arr(dW),
                                       self._arr(ws), sizes, self.n, stream), "asi_wgrad_batched")


def perplexity(dW, dW_approx, n, out, ws, ws_bytes, stream=0):
    """asi_perplexity: ||dW - dW_approx||_F into the device double `out`."""
    _check(lib().asi_perplexity(dW, dW_approx, int(n), out, ws, ws_bytes, stream), "asi_perplexity")


def gaussian_stream(seed, stream_id, n, out, stream=0):
    """asi_gaussian_stream: the first n values of the N(0, 1) stream (seed, stream_id) into device fp32 `out`."""
    _check(lib().asi_gaussian_stream(int(seed), int(stream_id), int(n), out, stream), "asi_gaussian_stream")


def philox_words(seed, stream_id, n_groups, out, stream=0):
    """asi_philox_words: the raw words of the first n_groups groups into device uint32 `out` (4 per group)."""
    _check(lib().asi_philox_words(int(seed), int(stream_id), int(n_groups), out, stream), "asi_philox_words")


def perplexity_ws_bytes():
    return lib().asi_perplexity_ws_bytes()


KERNEL_IDS = {"modeprod": 1, "expand": 2, "qr": 3, "conv_tail": 4, "sm_pass1": 5, "sm_core": 6,
              "sm_wgrad": 7}


def profile_begin(kernel_id: int, event_handles):
    """event_handles: flat list of CUDA event handles, [begin0, end0, begin1, end1, ...]."""
    n = len(event_handles) // 2
    arr = (C.c_void_p * (2 * n))(*event_handles)
    _check(lib().asi_profile_begin(int(kernel_id), arr, n), "asi_profile_begin")
    return arr            # keep alive until profile_end


def profile_end():
    b = C.c_double(0.0)
    n = lib().asi_profile_end(C.byref(b))
    return n, b.value
