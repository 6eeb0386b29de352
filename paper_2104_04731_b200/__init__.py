"""Python binding of libb2conv (argument marshalling only; every step runs in the CUDA library).

The functions mirror the C ABI in ``include/b2conv.h`` one to one.  Tensors are ``torch`` CUDA
tensors (used for device memory and streams only) or, for the ``*_host`` call, numpy arrays.
There is no fallback: if the shared library is missing, ``load()`` raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
# B2C_DEBUG_LIB=1 selects the debug build (bounds-checked kernels, guard bands round the workspace)
LIB_PATH = os.path.join(_HERE, "libb2conv_debug.so" if os.environ.get("B2C_DEBUG_LIB") == "1" else "libb2conv.so")

OK = 0
E_INVALID_ARG, E_UNSUPPORTED, E_WORKSPACE_TOO_SMALL, E_CUDA, E_TIMEOUT, E_NOT_READY, E_BOUNDS = -1, -2, -3, -4, -5, -6, -7
LAYOUT_NCHW, LAYOUT_NHWC = 0, 1
OUT_I32, OUT_I8 = 1, 2
AXIS_NPQ, AXIS_K, AXIS_C, AXIS_CRS, AXIS_SC, AXIS_C_PHASES = 1, 2, 3, 4, 5, 6
VARIANT_CP_TMA, VARIANT_IM2COL_EXPLICIT, VARIANT_IM2COL_GATHER, VARIANT_IM2COL_STAGED = 0, 1, 2, 3
VARIANT_ROW_UNROLL, VARIANT_SPACE_TO_DEPTH, VARIANT_DILATION_PACK = 4, 5, 6
VARIANT_CP_SHIFT, VARIANT_S2D_SHIFT, VARIANT_ROWPHASE_SHIFT, VARIANT_IM2COL_WINDOW = 7, 8, 9, 10
POLICY_AUTO_TIMED, POLICY_MIN_OVERHEAD, POLICY_MIN_WORKSPACE, POLICY_AUTO_TIMED_CONCURRENT = -1, -2, -3, -4
VARIANT_NAMES = {0: "channel_pack_tma_im2col", 1: "im2col_explicit", 2: "im2col_gather", 3: "im2col_staged_window",
                 4: "row_unroll_tma", 5: "space_to_depth_tma", 6: "dilation_phase_pack_tma",
                 7: "channel_pack_shift", 8: "space_to_depth_shift", 9: "row_phase_unroll_shift", 10: "im2col_tma_window"}

EXPORTS = [
    "b2c_out_shape", "b2c_enumerate", "b2c_plan_create", "b2c_plan_info", "b2c_plan_workspace_bytes",
    "b2c_plan_set_weights", "b2c_conv2d_int8_run", "b2c_conv2d_int8", "b2c_conv2d_int8_host",
    "b2c_plan_rewrite_activations", "b2c_conv2d_int8_run_rewritten", "b2c_plan_footprint", "b2c_plan_set_activation",
    "b2c_plan_create_grouped", "b2c_plan_create_grouped_timed", "b2c_plan_run_host_async", "b2c_plan_host_sync",
    "b2c_plan_device_status", "b2c_selftest_bounded_wait", "b2c_plan_destroy", "b2c_pack_activations", "b2c_im2col", "b2c_im2col_noalloc",
    "b2c_status_string",
    "b2c_last_cuda_error", "b2c_oneshot_status", "b2c_oneshot_cache_clear", "b2c_test_fail_nth_encode", "b2c_selftest_pack_wait", "b2c_measure_mma_rate", "b2c_measure_mma_rate_pair", "b2c_debug_build", "b2c_plan_debug_info",
    "b2c_plan_check_canaries", "b2c_test_shrink_checked_ranges",
]


class ConvDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "N", "C", "H", "W", "K", "R", "S", "stride_h", "stride_w", "pad_h", "pad_w", "dil_h", "dil_w",
        "shift", "in_layout", "out_layout", "out_mode")]


class Embedding(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("id", "map_m", "map_n", "map_k", "variant", "tile_m", "tile_n", "split_k")] + [
        ("o_mac", ctypes.c_int64), ("o_data", ctypes.c_int64), ("workspace_bytes", ctypes.c_int64),
        ("device_us", ctypes.c_float)]

    def as_dict(self):
        d = {n: getattr(self, n) for n, _ in self._fields_}
        d["variant_name"] = VARIANT_NAMES.get(self.variant, "?")
        return d


class B2CError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = _lib.b2c_status_string(code).decode() if _lib is not None else str(code)
        extra = ""
        if code == E_CUDA and _lib is not None:
            extra = " (cuda error %d)" % _lib.b2c_last_cuda_error()
        super().__init__("%s: %s%s" % (where, msg, extra))


_lib = None


def load():
    """Loads libb2conv.so; raises if it has not been built (no fallback path exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "libb2conv.so is missing: build it with `python -m paper_2104_04731_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    i32, vp = ctypes.c_int, ctypes.c_void_p
    pd, pe = ctypes.POINTER(ConvDesc), ctypes.POINTER(Embedding)
    pi32 = ctypes.POINTER(ctypes.c_int32)
    lib.b2c_out_shape.argtypes = [pd, pi32, pi32]
    lib.b2c_enumerate.argtypes = [pd, pe, ctypes.c_int32, pi32]
    lib.b2c_plan_create.argtypes = [pd, ctypes.c_int32, vp, ctypes.POINTER(vp)]
    lib.b2c_plan_info.argtypes = [vp, pe]
    lib.b2c_plan_workspace_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
    lib.b2c_plan_set_weights.argtypes = [vp, vp, vp]
    lib.b2c_conv2d_int8_run.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.b2c_plan_rewrite_activations.argtypes = [vp, vp, vp, vp]
    lib.b2c_conv2d_int8_run_rewritten.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.b2c_plan_set_activation.argtypes = [vp, vp, i32, vp]
    lib.b2c_plan_create_grouped.argtypes = [pd, ctypes.c_int32, ctypes.POINTER(vp)]
    lib.b2c_plan_create_grouped_timed.argtypes = [pd, ctypes.c_int32, vp, ctypes.POINTER(vp)]
    lib.b2c_plan_footprint.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
    lib.b2c_conv2d_int8.argtypes = [i32] * 11 + [vp] * 5
    lib.b2c_conv2d_int8_host.argtypes = [i32] * 11 + [vp] * 4
    lib.b2c_plan_run_host_async.argtypes = [vp, vp, vp, vp]
    lib.b2c_plan_host_sync.argtypes = [vp]
    lib.b2c_plan_device_status.argtypes = [vp, pi32]
    lib.b2c_plan_destroy.argtypes = [vp]
    lib.b2c_selftest_bounded_wait.argtypes = [vp, vp]
    lib.b2c_selftest_pack_wait.argtypes = [vp, vp]
    lib.b2c_plan_destroy.restype = None
    lib.b2c_pack_activations.argtypes = [vp, vp] + [i32] * 5 + [vp]
    lib.b2c_im2col.argtypes = [pd, vp, vp, i32, vp]
    lib.b2c_im2col_noalloc.argtypes = [pd, vp, vp, i32, vp]
    lib.b2c_status_string.argtypes = [i32]
    lib.b2c_status_string.restype = ctypes.c_char_p
    lib.b2c_last_cuda_error.argtypes = []
    lib.b2c_oneshot_status.argtypes = [pi32]
    lib.b2c_debug_build.argtypes = []
    lib.b2c_plan_debug_info.argtypes = [vp, pi32, ctypes.POINTER(ctypes.c_int64)]
    lib.b2c_plan_check_canaries.argtypes = [vp, vp, pi32]
    lib.b2c_test_shrink_checked_ranges.argtypes = [ctypes.c_longlong]
    lib.b2c_measure_mma_rate.argtypes = [i32, i32, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float), vp]
    lib.b2c_measure_mma_rate_pair.argtypes = [i32, i32, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float), vp]
    lib.b2c_oneshot_cache_clear.argtypes = []
    lib.b2c_test_fail_nth_encode.argtypes = [i32]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("b2c_plan_destroy", "b2c_status_string"):
            fn.restype = ctypes.c_int
    _lib = lib
    return lib


def _check(code: int, where: str):
    if code != OK:
        raise B2CError(code, where)


def _pair(v) -> Tuple[int, int]:
    if isinstance(v, (tuple, list)):
        return int(v[0]), int(v[1])
    return int(v), int(v)


def make_desc(N, C, H, W, K, R, S, stride=1, pad=0, dilation=1, shift=0, in_layout=LAYOUT_NCHW,
              out_layout=LAYOUT_NCHW, out_mode=OUT_I32) -> ConvDesc:
    sh, sw = _pair(stride)
    ph, pw = _pair(pad)
    dh, dw = _pair(dilation)
    return ConvDesc(N, C, H, W, K, R, S, sh, sw, ph, pw, dh, dw, shift, in_layout, out_layout, out_mode)


def status_string(code: int) -> str:
    return load().b2c_status_string(code).decode()


def out_shape(desc: ConvDesc) -> Tuple[int, int]:
    P, Q = ctypes.c_int32(), ctypes.c_int32()
    _check(load().b2c_out_shape(ctypes.byref(desc), ctypes.byref(P), ctypes.byref(Q)), "b2c_out_shape")
    return P.value, Q.value


def enumerate_embeddings(desc: ConvDesc) -> List[Embedding]:
    lib = load()
    n = ctypes.c_int32()
    _check(lib.b2c_enumerate(ctypes.byref(desc), None, 0, ctypes.byref(n)), "b2c_enumerate")
    arr = (Embedding * n.value)()
    _check(lib.b2c_enumerate(ctypes.byref(desc), arr, n.value, ctypes.byref(n)), "b2c_enumerate")
    return list(arr)


def _stream_ptr(stream=None):
    import torch

    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _dptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


class Plan:
    """Owns a ``b2c_plan``.  ``run`` enqueues the whole path on the current torch stream."""

    def __init__(self, desc: ConvDesc, policy_or_id: int = POLICY_MIN_OVERHEAD, stream=None, groups: int = 1):
        """groups > 1: grouped convolution (desc.C and desc.K are the totals, weights [K, C/groups, R, S]); with a
        timed policy the form (in place, or all groups merged into a dense convolution) is chosen by timing."""
        self._lib = load()
        self.desc = desc
        h = ctypes.c_void_p()
        if groups > 1 and policy_or_id in (POLICY_AUTO_TIMED, POLICY_AUTO_TIMED_CONCURRENT):
            _check(self._lib.b2c_plan_create_grouped_timed(ctypes.byref(desc), groups, _stream_ptr(stream), ctypes.byref(h)),
                   "b2c_plan_create_grouped_timed")
        elif groups > 1:
            _check(self._lib.b2c_plan_create_grouped(ctypes.byref(desc), groups, ctypes.byref(h)), "b2c_plan_create_grouped")
        else:
            _check(self._lib.b2c_plan_create(ctypes.byref(desc), policy_or_id, _stream_ptr(stream), ctypes.byref(h)),
                   "b2c_plan_create")
        self._h = h

    def info(self) -> Embedding:
        e = Embedding()
        _check(self._lib.b2c_plan_info(self._h, ctypes.byref(e)), "b2c_plan_info")
        return e

    def workspace_bytes(self) -> int:
        n = ctypes.c_size_t()
        _check(self._lib.b2c_plan_workspace_bytes(self._h, ctypes.byref(n)), "b2c_plan_workspace_bytes")
        return n.value

    def set_weights(self, w, stream=None):
        _check(self._lib.b2c_plan_set_weights(self._h, _dptr(w), _stream_ptr(stream)), "b2c_plan_set_weights")

    def run(self, x, y32=None, y8=None, workspace=None, stream=None):
        _check(self._lib.b2c_conv2d_int8_run(self._h, _dptr(x), _dptr(y32), _dptr(y8), _dptr(workspace),
                                              _stream_ptr(stream)), "b2c_conv2d_int8_run")

    def set_activation(self, bias=None, relu=False, stream=None):
        """Activation step before the outputs are written: int32 CUDA tensor `bias` [K] (or None), ReLU flag."""
        _check(self._lib.b2c_plan_set_activation(self._h, _dptr(bias), int(bool(relu)), _stream_ptr(stream)),
               "b2c_plan_set_activation")

    def rewrite_activations(self, x, workspace=None, stream=None):
        """Only the layout rewrite of x into the workspace (the "Transf." half of run)."""
        _check(self._lib.b2c_plan_rewrite_activations(self._h, _dptr(x), _dptr(workspace), _stream_ptr(stream)),
               "b2c_plan_rewrite_activations")

    def run_rewritten(self, x, y32=None, y8=None, workspace=None, stream=None):
        """Only the MMA kernel, epilogue and split finish on an already rewritten workspace (the "Op." half)."""
        _check(self._lib.b2c_conv2d_int8_run_rewritten(self._h, _dptr(x), _dptr(y32), _dptr(y8), _dptr(workspace),
                                                        _stream_ptr(stream)), "b2c_conv2d_int8_run_rewritten")

    def run_host_async(self, x, y32=None, y8=None):
        """Streaming call on numpy HOST arrays (page-locked for overlap): enqueues copy in, the whole path and
        copy out, and returns; up to three calls are in flight.  The arrays stay untouched until host_sync()."""
        def hp(a):
            return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None

        _check(self._lib.b2c_plan_run_host_async(self._h, hp(x), hp(y32), hp(y8)), "b2c_plan_run_host_async")

    def host_sync(self):
        """Waits until every run_host_async of this plan has delivered its outputs."""
        _check(self._lib.b2c_plan_host_sync(self._h), "b2c_plan_host_sync")

    def footprint(self) -> Tuple[int, int]:
        """(bytes of the rewritten activation operand, bytes of the packed weights)."""
        a, b = ctypes.c_size_t(), ctypes.c_size_t()
        _check(self._lib.b2c_plan_footprint(self._h, ctypes.byref(a), ctypes.byref(b)), "b2c_plan_footprint")
        return a.value, b.value

    def device_status(self) -> int:
        s = ctypes.c_int32()
        _check(self._lib.b2c_plan_device_status(self._h, ctypes.byref(s)), "b2c_plan_device_status")
        return s.value

    def selftest_bounded_wait(self, stream=None):
        """Enqueues the bounded-wait self-test; afterwards device_status() reports E_TIMEOUT once."""
        _check(self._lib.b2c_selftest_bounded_wait(self._h, _stream_ptr(stream)), "b2c_selftest_bounded_wait")

    def debug_info(self) -> Tuple[int, int]:
        """(site, byte offset) of the out-of-range access the last device_status() reported (debug build)."""
        site, off = ctypes.c_int32(), ctypes.c_int64()
        _check(self._lib.b2c_plan_debug_info(self._h, ctypes.byref(site), ctypes.byref(off)), "b2c_plan_debug_info")
        return site.value, off.value

    def canaries_intact(self, workspace) -> bool:
        """Debug build: True if the guard bands round `workspace` are untouched."""
        ok = ctypes.c_int32()
        _check(self._lib.b2c_plan_check_canaries(self._h, _dptr(workspace), ctypes.byref(ok)), "b2c_plan_check_canaries")
        return bool(ok.value)

    def selftest_pack_wait(self, stream=None):
        """The same self-test for the activation-pack kernel's wait on its bulk copies."""
        _check(self._lib.b2c_selftest_pack_wait(self._h, _stream_ptr(stream)), "b2c_selftest_pack_wait")

    def destroy(self):
        if getattr(self, "_h", None):
            self._lib.b2c_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def conv2d_int8(x, w, stride=1, pad=0, dilation=1, shift=0, y32=None, y8=None, stream=None):
    """One-shot call on CUDA tensors: x int8 [N,C,H,W], w int8 [K,C,R,S]; writes y32 / y8 ([N,K,P,Q])."""
    N, C, H, W = x.shape
    K, _, R, S = w.shape
    _check(load().b2c_conv2d_int8(N, C, H, W, K, R, S, stride, pad, dilation, shift, _dptr(x), _dptr(w), _dptr(y32),
                                  _dptr(y8), _stream_ptr(stream)), "b2c_conv2d_int8")


def measure_mma_rate(tile_n: int = 256, mmas_per_block: int = 20000, stream=None):
    """(device_us, cycles_per_mma) of back-to-back 128 x tile_n x 32 int8 MMAs on all SMs, operands in shared memory."""
    us, cyc = ctypes.c_float(), ctypes.c_float()
    _check(load().b2c_measure_mma_rate(tile_n, mmas_per_block, ctypes.byref(us), ctypes.byref(cyc), _stream_ptr(stream)),
           "b2c_measure_mma_rate")
    return us.value, cyc.value


def measure_mma_rate_pair(tile_n: int = 256, mmas_per_pair: int = 20000, stream=None):
    """(device_us, cycles_per_mma) of back-to-back two-SM 256 x tile_n x 32 int8 MMAs on all 74 block pairs."""
    us, cyc = ctypes.c_float(), ctypes.c_float()
    _check(load().b2c_measure_mma_rate_pair(tile_n, mmas_per_pair, ctypes.byref(us), ctypes.byref(cyc), _stream_ptr(stream)),
           "b2c_measure_mma_rate_pair")
    return us.value, cyc.value


def debug_build() -> bool:
    return bool(load().b2c_debug_build())


def test_shrink_checked_ranges(nbytes: int):
    """Debug-build test hook: declare every checked range `nbytes` shorter than it is (0 restores)."""
    _check(load().b2c_test_shrink_checked_ranges(nbytes), "b2c_test_shrink_checked_ranges")


def oneshot_status() -> int:
    """Status of the one-shot cache on the current device (E_TIMEOUT once after a bounded wait expired)."""
    s = ctypes.c_int32()
    _check(load().b2c_oneshot_status(ctypes.byref(s)), "b2c_oneshot_status")
    return s.value


def oneshot_cache_clear():
    """Frees the plans and scratch the one-shot calls cached on the current device."""
    _check(load().b2c_oneshot_cache_clear(), "b2c_oneshot_cache_clear")


def test_fail_nth_encode(n: int):
    """Host-side fault injection: the n-th tensor-map encode from now on fails (0 disarms)."""
    _check(load().b2c_test_fail_nth_encode(n), "b2c_test_fail_nth_encode")


def conv2d_int8_host(x, w, stride=1, pad=0, dilation=1, shift=0, y32=None, y8=None):
    """One-shot call on numpy host arrays (copies in, runs, copies out, synchronises)."""
    N, C, H, W = x.shape
    K, _, R, S = w.shape

    def hp(a):
        return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None

    _check(load().b2c_conv2d_int8_host(N, C, H, W, K, R, S, stride, pad, dilation, shift, hp(x), hp(w), hp(y32),
                                       hp(y8)), "b2c_conv2d_int8_host")


def pack_activations(x, out, C_pad: int, stream=None):
    N, C, H, W = x.shape
    _check(load().b2c_pack_activations(_dptr(x), _dptr(out), N, C, H, W, C_pad, _stream_ptr(stream)),
           "b2c_pack_activations")


def im2col(desc: ConvDesc, x, a, K_pad: int, stream=None):
    _check(load().b2c_im2col(ctypes.byref(desc), _dptr(x), _dptr(a), K_pad, _stream_ptr(stream)), "b2c_im2col")


def im2col_noalloc(desc: ConvDesc, x, a, K_pad: int, stream=None):
    """Same result as ``im2col`` without any device allocation inside the library (fixed 128 KB
    table, K_pad <= 16384); for callers that run where cudaMalloc is off limits.  Calls that may
    overlap on the GPU must be ordered by the caller."""
    _check(load().b2c_im2col_noalloc(ctypes.byref(desc), _dptr(x), _dptr(a), K_pad, _stream_ptr(stream)),
           "b2c_im2col_noalloc")
