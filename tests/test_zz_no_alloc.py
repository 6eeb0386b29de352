"""The allocation-free stencil unroll (b2c_im2col_noalloc) against the allocating entry point.

Some users of this library run where device allocation is not allowed (a framework region frozen
against cudaMalloc, a latency-critical loop, a process whose memory all belongs to another pool).
They get the same matrix from a call that keeps its lookup table in a fixed array inside the
library.  The table is shared by all calls and keeps what the last call wrote, so this test makes
two calls in a row with different geometries (the second one shorter, so that stale entries of the
first would show) and compares each, byte for byte, with b2c_im2col and with the CPU oracle's
stencil-unroll matrix.  The file name makes pytest collect it last.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2104_04731_b200 as b2c
from paper_2104_04731_b200.synth import int8_uniform

pytestmark = pytest.mark.gpu


def _both(lib, geom, in_layout, seed):
    N, C, H, W, R, S, stride, pad, dil = geom
    x = int8_uniform((N, C, H, W), seed)
    xin = x if in_layout == 0 else np.ascontiguousarray(x.transpose(0, 2, 3, 1))
    xd = torch.from_numpy(np.ascontiguousarray(xin)).cuda()
    d = lib.make_desc(N, C, H, W, 1, R, S, stride, pad, dil, in_layout=in_layout)
    P, Q = lib.out_shape(d)
    K_pad = -(-C * R * S // 32) * 32
    ref = torch.full((N * P * Q, K_pad), 55, dtype=torch.int8, device="cuda")
    got = torch.full((N * P * Q, K_pad), 66, dtype=torch.int8, device="cuda")
    lib.im2col(d, xd, ref, K_pad)          # existing entry point (allocates its table)
    lib.im2col_noalloc(d, xd, got, K_pad)  # the allocation-free one
    torch.cuda.synchronize()
    want = oracle.im2col(x, R, S, stride, pad, dil)   # [N*P*Q][C*R*S], from the CPU oracle
    return got.cpu().numpy(), ref.cpu().numpy(), want


def test_two_calls_in_a_row_match_the_allocating_entry_point(lib):
    first = (2, 16, 13, 11, 3, 5, (2, 1), (1, 2), (1, 2))   # C*R*S = 240 -> K_pad 256
    second = (1, 3, 20, 21, 7, 7, 2, 3, 1)                   # C*R*S = 147 -> K_pad 160 (shorter table)
    for i, (geom, in_layout) in enumerate([(first, 0), (second, 1)]):
        got, ref, want = _both(lib, geom, in_layout, 900 + i)
        assert np.array_equal(got, ref), "call %d differs from b2c_im2col" % (i + 1)
        assert np.array_equal(got[:, :want.shape[1]], want), "call %d differs from the oracle" % (i + 1)
        assert not got[:, want.shape[1]:].any()


def test_size_limit_is_reported_without_launching(lib):
    # C*R*S = 17408 needs a table of 17408 entries: beyond the fixed array
    d = lib.make_desc(1, 17408, 2, 2, 1, 1, 1)
    x = torch.zeros(17408 * 4, dtype=torch.int8, device="cuda")
    a = torch.zeros(4 * 17408, dtype=torch.int8, device="cuda")
    rc = lib.load().b2c_im2col_noalloc(ctypes.byref(d), ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(a.data_ptr()),
                                       17408, None)
    assert rc == b2c.E_WORKSPACE_TOO_SMALL
    rc = lib.load().b2c_im2col_noalloc(None, None, None, 32, None)
    assert rc == b2c.E_INVALID_ARG
