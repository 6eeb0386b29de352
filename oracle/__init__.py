"""CPU oracle (test infrastructure only).

Thin ctypes front end over ``conv_oracle.c``: the plain seven-loop int8 convolution with int32
range check and shift/clip requantisation, plus the separate stencil-unroll + GEMM path used to
cross-check it.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the GPU library never does, and this package never imports the GPU library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "conv_oracle.c")
_SO = os.path.join(_HERE, "liboracle_conv.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile conv_oracle.c with gcc (OpenMP) into liboracle_conv.so next to it."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC]
        )
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_void_p
        lib.oracle_out_extent.argtypes = [i32] * 5
        lib.oracle_out_extent.restype = i32
        lib.oracle_requant.argtypes = [i64, i32]
        lib.oracle_requant.restype = ctypes.c_int8
        lib.oracle_conv2d_int8.argtypes = [vp, vp] + [i32] * 14 + [vp, vp, i32]
        lib.oracle_conv2d_int8.restype = i32
        lib.oracle_conv2d_int8_act.argtypes = [vp, vp, vp, i32] + [i32] * 14 + [vp, vp, i32]
        lib.oracle_conv2d_int8_act.restype = i32
        lib.oracle_conv2d_int8_grouped.argtypes = [vp, vp, vp, i32, i32] + [i32] * 14 + [vp, vp, i32]
        lib.oracle_conv2d_int8_grouped.restype = i32
        lib.oracle_im2col.argtypes = [vp] + [i32] * 12 + [vp]
        lib.oracle_im2col.restype = None
        lib.oracle_gemm_abt.argtypes = [vp, vp, i64, i64, i64, vp]
        lib.oracle_gemm_abt.restype = None
        lib.oracle_pack_nhwc_cpad.argtypes = [vp] + [i32] * 5 + [vp]
        lib.oracle_pack_nhwc_cpad.restype = None
        _lib = lib
    return _lib


def _pair(v):
    if isinstance(v, (tuple, list)):
        return int(v[0]), int(v[1])
    return int(v), int(v)


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def out_extent(size: int, k: int, stride: int, pad: int, dil: int) -> int:
    return int(_load().oracle_out_extent(size, k, stride, pad, dil))


def out_shape(H, W, R, S, stride=1, pad=0, dilation=1):
    sh, sw = _pair(stride)
    ph, pw = _pair(pad)
    dh, dw = _pair(dilation)
    return out_extent(H, R, sh, ph, dh), out_extent(W, S, sw, pw, dw)


def requant(acc: int, shift: int) -> int:
    return int(_load().oracle_requant(int(acc), int(shift)))


def conv2d_int8(x, w, stride=1, pad=0, dilation=1, shift=0, want_i32=True, want_i8=True, threads=0, bias=None,
                relu=False, groups=1):
    """x: int8 [N,C,H,W]; w: int8 [K,C,R,S] -> (y32 int32 [N,K,P,Q] or None, y8 int8 or None).

    `groups` > 1: grouped convolution, w is [K, C/groups, R, S] (groups = C = K: depth-wise).
    Optional activation step before the outputs are written: per-output-channel int32 `bias` [K]
    added to the exact sum, then ReLU.  Raises OverflowError when a value leaves the int32 range.
    """
    x = np.ascontiguousarray(x, dtype=np.int8)
    w = np.ascontiguousarray(w, dtype=np.int8)
    N, C, H, W = x.shape
    K, C2, R, S = w.shape
    groups = int(groups)
    assert groups >= 1 and C % groups == 0 and K % groups == 0 and C2 * groups == C  # w is [K][C/groups][R][S]
    sh, sw = _pair(stride)
    ph, pw = _pair(pad)
    dh, dw = _pair(dilation)
    P, Q = out_shape(H, W, R, S, (sh, sw), (ph, pw), (dh, dw))
    y32 = np.empty((N, K, P, Q), dtype=np.int32) if want_i32 else None
    y8 = np.empty((N, K, P, Q), dtype=np.int8) if want_i8 else None
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.int32)
        assert bias.shape == (K,)
    rc = _load().oracle_conv2d_int8_grouped(
        _ptr(x), _ptr(w), _ptr(bias), int(bool(relu)), groups, N, C, H, W, K, R, S, sh, sw, ph, pw, dh, dw, int(shift),
        _ptr(y32), _ptr(y8), int(threads)
    )
    if rc != 0:
        raise OverflowError("an accumulator left the int32 range")
    return y32, y8


def im2col(x, R, S, stride=1, pad=0, dilation=1):
    """Stencil unroll: int8 [N,C,H,W] -> int8 [N*P*Q, C*R*S] (reduction order c, r, s)."""
    x = np.ascontiguousarray(x, dtype=np.int8)
    N, C, H, W = x.shape
    sh, sw = _pair(stride)
    ph, pw = _pair(pad)
    dh, dw = _pair(dilation)
    P, Q = out_shape(H, W, R, S, (sh, sw), (ph, pw), (dh, dw))
    A = np.empty((N * P * Q, C * R * S), dtype=np.int8)
    _load().oracle_im2col(_ptr(x), N, C, H, W, R, S, sh, sw, ph, pw, dh, dw, _ptr(A))
    return A


def gemm_abt(A, B):
    """D[m][j] = sum_z A[m][z] * B[j][z], int64."""
    A = np.ascontiguousarray(A, dtype=np.int8)
    B = np.ascontiguousarray(B, dtype=np.int8)
    M, Kg = A.shape
    Nn, Kg2 = B.shape
    assert Kg == Kg2
    D = np.empty((M, Nn), dtype=np.int64)
    _load().oracle_gemm_abt(_ptr(A), _ptr(B), M, Nn, Kg, _ptr(D))
    return D


def conv2d_via_im2col_gemm(x, w, stride=1, pad=0, dilation=1):
    """The GEMM view of the convolution (stencil unroll, then C += A * B^T): int64 [N,K,P,Q]."""
    N, C, H, W = x.shape
    K, _, R, S = w.shape
    P, Q = out_shape(H, W, R, S, stride, pad, dilation)
    A = im2col(x, R, S, stride, pad, dilation)
    D = gemm_abt(A, np.ascontiguousarray(w).reshape(K, C * R * S))
    return np.ascontiguousarray(D.reshape(N, P, Q, K).transpose(0, 3, 1, 2))


def pack_nhwc_cpad(x, C_pad):
    """NCHW int8 -> NHWC int8 with channels zero-padded to C_pad."""
    x = np.ascontiguousarray(x, dtype=np.int8)
    N, C, H, W = x.shape
    out = np.empty((N, H, W, C_pad), dtype=np.int8)
    _load().oracle_pack_nhwc_cpad(_ptr(x), N, C, H, W, int(C_pad), _ptr(out))
    return out
