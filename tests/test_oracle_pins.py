"""Pins for the CPU oracle: every check here compares oracle/ against something fixed by the
mathematics (brute force written differently, textbook special cases, closed forms, hand
tables), never against the GPU path and never against the oracle's own formula."""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2104_04731_b200.synth import CONFIGS, int8_uniform

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def scatter_conv(x, w, stride, pad, dil):
    """Second evaluator, structured the other way round: walk over *input* pixels and taps and
    scatter each product into the output it belongs to (pure Python, tiny shapes only)."""
    N, C, H, W = x.shape
    K, _, R, S = w.shape
    sh, sw = stride
    ph, pw = pad
    dh, dw = dil
    P = (H + 2 * ph - dh * (R - 1) - 1) // sh + 1 if H + 2 * ph - dh * (R - 1) - 1 >= 0 else 0
    Q = (W + 2 * pw - dw * (S - 1) - 1) // sw + 1 if W + 2 * pw - dw * (S - 1) - 1 >= 0 else 0
    y = np.zeros((N, K, max(P, 0), max(Q, 0)), dtype=np.int64)
    for n, c, h, ww in itertools.product(range(N), range(C), range(H), range(W)):
        xv = int(x[n, c, h, ww])
        for r, s in itertools.product(range(R), range(S)):
            # input pixel (h, ww) is tap (r, s) of output (p, q) iff h = p*sh - ph + r*dh
            tp, tq = h + ph - r * dh, ww + pw - s * dw
            if tp < 0 or tq < 0 or tp % sh or tq % sw:
                continue
            p, q = tp // sh, tq // sw
            if p >= P or q >= Q:
                continue
            for k in range(K):
                y[n, k, p, q] += xv * int(w[k, c, r, s])
    return y


# ---- P0: hand-worked example ------------------------------------------------------------------
def _read_vec(path, key):
    for line in open(path):
        if line.startswith(key + " "):
            return [int(t) for t in line.split()[1:]]
    raise KeyError(key)


def test_hand_worked_example():
    f = os.path.join(GOLDEN, "hand_conv_3x3.txt")
    x = np.array(_read_vec(f, "x"), dtype=np.int8).reshape(1, 1, 3, 3)
    w = np.array(_read_vec(f, "w"), dtype=np.int8).reshape(1, 1, 2, 2)
    y = np.array(_read_vec(f, "y"), dtype=np.int32).reshape(1, 1, 4, 4)
    y32, _ = oracle.conv2d_int8(x, w, stride=1, pad=1)
    assert np.array_equal(y32, y)


# ---- P1: brute force on tiny inputs -------------------------------------------------------------
@pytest.mark.parametrize("stride", [(1, 1), (2, 2), (3, 2), (1, 3)])
@pytest.mark.parametrize("pad", [(0, 0), (1, 1), (2, 1), (0, 2)])
@pytest.mark.parametrize("dil", [(1, 1), (2, 2), (1, 2)])
def test_brute_force_scatter(stride, pad, dil):
    shapes = [(2, 3, 6, 5, 4, 3, 2), (1, 2, 5, 6, 3, 2, 3), (1, 1, 4, 4, 2, 1, 1)]
    for i, (N, C, H, W, K, R, S) in enumerate(shapes):
        x = int8_uniform((N, C, H, W), 11 + i)
        w = int8_uniform((K, C, R, S), 21 + i)
        ref = scatter_conv(x, w, stride, pad, dil)
        P, Q = oracle.out_shape(H, W, R, S, stride, pad, dil)
        assert (P, Q) == ref.shape[2:]
        if P == 0 or Q == 0:
            continue
        y32, _ = oracle.conv2d_int8(x, w, stride, pad, dil)
        assert np.array_equal(y32.astype(np.int64), ref)


def test_out_extent_values():
    # (in, k, stride, pad, dil) -> extent; values worked by hand from the floor formula
    table = {(14, 3, 1, 1, 1): 14, (56, 3, 1, 1, 1): 56, (224, 7, 2, 3, 1): 112, (96, 9, 2, 0, 1): 44,
             (480, 21, 2, 0, 1): 230, (14, 3, 2, 1, 1): 7, (5, 3, 1, 0, 2): 1, (4, 3, 1, 0, 2): 0,
             (7, 3, 3, 0, 1): 2, (1, 1, 1, 0, 1): 1}
    for args, want in table.items():
        assert oracle.out_extent(*args) == want


# ---- P2: 1x1, stride 1, no pad == matrix multiply ---------------------------------------------------
def test_pointwise_is_matmul():
    x = int8_uniform((3, 37, 5, 7), 31)
    w = int8_uniform((19, 37, 1, 1), 32)
    y32, _ = oracle.conv2d_int8(x, w)
    ref = np.einsum("kc,nchw->nkhw", w[:, :, 0, 0].astype(np.int64), x.astype(np.int64))
    assert np.array_equal(y32.astype(np.int64), ref)


# ---- P3: delta kernel == shifted, subsampled copy ------------------------------------------------
@pytest.mark.parametrize("stride,pad,dil", [(1, 0, 1), (1, 2, 1), (2, 1, 1), (2, 3, 2), (3, 1, 2)])
def test_delta_kernel_is_shift(stride, pad, dil):
    N, C, H, W, K, R, S = 2, 3, 9, 11, 4, 3, 4
    x = int8_uniform((N, C, H, W), 41)
    for (k0, c0, r0, s0) in [(0, 0, 0, 0), (1, 2, 2, 3), (3, 1, 1, 2)]:
        w = np.zeros((K, C, R, S), dtype=np.int8)
        w[k0, c0, r0, s0] = 1
        y32, _ = oracle.conv2d_int8(x, w, stride, pad, dil)
        P, Q = y32.shape[2:]
        xp = np.zeros((N, H + 2 * pad + 64, W + 2 * pad + 64), dtype=np.int32)
        xp[:, pad:pad + H, pad:pad + W] = x[:, c0]
        want = xp[:, r0 * dil:, s0 * dil:][:, ::stride, ::stride][:, :P, :Q]
        assert np.array_equal(y32[:, k0], want)
        others = [k for k in range(K) if k != k0]
        assert not y32[:, others].any()


# ---- P4: linearity --------------------------------------------------------------------------------
def test_linearity_in_weights_and_input():
    x = int8_uniform((2, 5, 8, 9), 51)
    w1 = (int8_uniform((6, 5, 3, 3), 52) // 2).astype(np.int8)
    w2 = (int8_uniform((6, 5, 3, 3), 53) // 2).astype(np.int8)
    a, _ = oracle.conv2d_int8(x, w1, 2, 1)
    b, _ = oracle.conv2d_int8(x, w2, 2, 1)
    c, _ = oracle.conv2d_int8(x, (w1.astype(np.int16) + w2).astype(np.int8), 2, 1)
    assert np.array_equal(a + b, c)
    x1 = (x // 2).astype(np.int8)
    x2 = (int8_uniform(x.shape, 54) // 2).astype(np.int8)
    a, _ = oracle.conv2d_int8(x1, w1, 1, 1)
    b, _ = oracle.conv2d_int8(x2, w1, 1, 1)
    c, _ = oracle.conv2d_int8((x1.astype(np.int16) + x2).astype(np.int8), w1, 1, 1)
    assert np.array_equal(a + b, c)


# ---- P5: closed form for constant tensors -----------------------------------------------------------
def _tap_count(p, stride, pad, dil, k, size):
    return sum(1 for r in range(k) if 0 <= p * stride - pad + r * dil < size)


@pytest.mark.parametrize("xv,wv", [(1, 1), (-128, -128), (127, -128)])
@pytest.mark.parametrize("geom", [(7, 9, 3, 3, 1, 1, 1), (8, 8, 3, 5, 2, 2, 1), (10, 6, 3, 2, 2, 3, 2), (6, 6, 7, 7, 2, 3, 1)])
def test_constant_closed_form(xv, wv, geom):
    H, W, R, S, stride, pad, dil = geom
    C, K, N = 5, 3, 2
    x = np.full((N, C, H, W), xv, dtype=np.int8)
    w = np.full((K, C, R, S), wv, dtype=np.int8)
    y32, _ = oracle.conv2d_int8(x, w, stride, pad, dil)
    P, Q = y32.shape[2:]
    for p in range(P):
        for q in range(Q):
            want = C * xv * wv * _tap_count(p, stride, pad, dil, R, H) * _tap_count(q, stride, pad, dil, S, W)
            assert (y32[:, :, p, q] == want).all()


# ---- P6: the GEMM view (stencil unroll + C += A.B^T), separate code path ---------------------------
@pytest.mark.parametrize("geom", [(2, 3, 12, 13, 5, 3, 3, 1, 1, 1), (1, 4, 9, 9, 6, 3, 2, 2, 0, 2), (2, 1, 10, 20, 4, 5, 7, 2, 0, 1)])
def test_im2col_gemm_path(geom):
    N, C, H, W, K, R, S, stride, pad, dil = geom
    x = int8_uniform((N, C, H, W), 61)
    w = int8_uniform((K, C, R, S), 62)
    y32, _ = oracle.conv2d_int8(x, w, stride, pad, dil)
    via = oracle.conv2d_via_im2col_gemm(x, w, stride, pad, dil)
    assert np.array_equal(y32.astype(np.int64), via)


def test_im2col_against_numpy_windows():
    # the unrolled matrix itself, against numpy's sliding windows on a zero-padded copy
    N, C, H, W, R, S, stride, pad, dil = 2, 3, 8, 9, 3, 2, 2, 1, 2
    x = int8_uniform((N, C, H, W), 63)
    A = oracle.im2col(x, R, S, stride, pad, dil)
    xp = np.pad(x, ((0, 0), (0, 0), (pad, pad), (pad, pad)))
    win = np.lib.stride_tricks.sliding_window_view(xp, (dil * (R - 1) + 1, dil * (S - 1) + 1), axis=(2, 3))
    win = win[:, :, ::stride, ::stride, ::dil, ::dil]  # n c p q r s
    want = win.transpose(0, 2, 3, 1, 4, 5).reshape(A.shape)
    assert np.array_equal(A, want)


def test_gemm_abt_is_matmul():
    A = int8_uniform((13, 29), 64)
    B = int8_uniform((7, 29), 65)
    assert np.array_equal(oracle.gemm_abt(A, B), A.astype(np.int64) @ B.astype(np.int64).T)


def test_pack_nhwc_cpad():
    x = int8_uniform((2, 5, 3, 4), 66)
    out = oracle.pack_nhwc_cpad(x, 16)
    assert np.array_equal(out[..., :5], x.transpose(0, 2, 3, 1))
    assert not out[..., 5:].any()


# ---- P7: requantisation hand table -----------------------------------------------------------------
def test_requant_table():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "requant_table.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) >= 20
    for acc, shift, want in rows:
        assert oracle.requant(int(acc), int(shift)) == int(want), (acc, shift)


def test_requant_inside_conv_matches_python_floor():
    x = int8_uniform((1, 16, 6, 6), 71)
    w = int8_uniform((8, 16, 3, 3), 72)
    for shift in (0, 1, 8, 31):
        y32, y8 = oracle.conv2d_int8(x, w, 1, 1, 1, shift)
        want = np.clip(y32.astype(np.int64) // (1 << shift), -128, 127)  # Python // is floor
        assert np.array_equal(y8.astype(np.int64), want)


# ---- P8: invariants ---------------------------------------------------------------------------------
def test_channel_permutation_and_zero_channel_padding():
    x = int8_uniform((2, 6, 7, 7), 81)
    w = int8_uniform((4, 6, 3, 3), 82)
    y, _ = oracle.conv2d_int8(x, w, 1, 1)
    perm = np.array([3, 0, 5, 1, 4, 2])
    y2, _ = oracle.conv2d_int8(x[:, perm], w[:, perm], 1, 1)
    assert np.array_equal(y, y2)
    xz = np.concatenate([x, np.zeros((2, 10, 7, 7), np.int8)], axis=1)
    wz = np.concatenate([w, int8_uniform((4, 10, 3, 3), 83)], axis=1)  # junk weights on zero channels
    y3, _ = oracle.conv2d_int8(xz, wz, 1, 1)
    assert np.array_equal(y, y3)
    assert np.abs(y.astype(np.int64)).max() <= 6 * 9 * 16384


def test_overflow_is_reported():
    # C*R*S*2^14 > 2^31 - 1 with all operands at -128 overflows int32
    C = 131073
    x = np.full((1, C, 1, 1), -128, dtype=np.int8)
    w = np.full((1, C, 1, 1), -128, dtype=np.int8)
    with pytest.raises(OverflowError):
        oracle.conv2d_int8(x, w)
    y, _ = oracle.conv2d_int8(x[:, :131071], w[:, :131071])
    assert int(y[0, 0, 0, 0]) == 131071 * 16384


# ---- the benchmark shapes: GEMM view agrees with the definition on sampled outputs ------------------
@pytest.mark.parametrize("cfg", CONFIGS[:4], ids=lambda c: c.name)
def test_config_samples_against_python(cfg):
    x, w = cfg.tensors()
    y32, y8 = oracle.conv2d_int8(x, w, cfg.stride, cfg.pad, cfg.dilation, cfg.shift)
    rng = np.random.default_rng(5)
    xi, wi = x.astype(np.int64), w.astype(np.int64)
    for _ in range(40):
        n, k, p, q = (int(rng.integers(0, d)) for d in y32.shape)
        acc = 0
        for r in range(cfg.R):
            for s in range(cfg.S):
                h, ww = p * cfg.stride - cfg.pad + r * cfg.dilation, q * cfg.stride - cfg.pad + s * cfg.dilation
                if 0 <= h < cfg.H and 0 <= ww < cfg.W:
                    acc += int(np.dot(xi[n, :, h, ww], wi[k, :, r, s]))
        assert int(y32[n, k, p, q]) == acc
        assert int(y8[n, k, p, q]) == max(-128, min(127, acc >> cfg.shift))  # Python >> on int is floor


@pytest.mark.parametrize("geom", [((2, 2), (2, 2)), ((4, 4), (4, 4)), ((2, 3), (1, 0)), ((3, 1), (0, 5))])
def test_dilated_conv_is_blown_up_stencil(geom):
    """Section 6.1 describes the reference for a dilated convolution as the same stencil "blown up
    with zeros": an undilated convolution whose kernel has the taps at (r*dil_h, s*dil_w) and zeros
    in between.  Pins the oracle's dilation handling against its own undilated path."""
    dil, pad = geom
    x = int8_uniform((2, 3, 15, 17), 71)
    w = int8_uniform((4, 3, 3, 2), 72)
    R, S = w.shape[2:]
    big = np.zeros((4, 3, dil[0] * (R - 1) + 1, dil[1] * (S - 1) + 1), dtype=np.int8)
    big[:, :, ::dil[0], ::dil[1]] = w
    got, _ = oracle.conv2d_int8(x, w, 1, pad, dil, 0)
    want, _ = oracle.conv2d_int8(x, big, 1, pad, 1, 0)
    assert got.shape == want.shape and np.array_equal(got, want)


def test_bias_and_relu_step():
    """Activation step (Section 5.1's vector unit; reading: per-channel int32 bias, then ReLU):
    pinned against numpy arithmetic on the plain convolution's int32 output, Python floor shift."""
    x = int8_uniform((2, 5, 9, 8), 81)
    w = int8_uniform((6, 5, 3, 3), 82)
    bias = np.array([0, 1, -1, 70000, -70000, 2 ** 20], dtype=np.int32)
    plain, _ = oracle.conv2d_int8(x, w, 1, 1, 1, 0)
    for relu in (False, True):
        for shift in (0, 4, 9):
            y32, y8 = oracle.conv2d_int8(x, w, 1, 1, 1, shift, bias=bias, relu=relu)
            t = plain.astype(np.int64) + bias.astype(np.int64)[None, :, None, None]
            if relu:
                t = np.maximum(t, 0)
            assert np.array_equal(y32, t)
            want8 = np.array([max(-128, min(127, int(v) >> shift)) for v in t.ravel()], dtype=np.int64).reshape(t.shape)
            assert np.array_equal(y8, want8)
            if relu:
                assert y32.min() == 0 and (plain + bias[None, :, None, None] < 0).any() and y8.min() >= 0
    # no bias, no ReLU is the plain convolution; a zero bias changes nothing
    a = oracle.conv2d_int8(x, w, 2, 0, 1, 3, bias=np.zeros(6, dtype=np.int32))
    b = oracle.conv2d_int8(x, w, 2, 0, 1, 3)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    # a bias that pushes a value past int32 is an error, not a wrap
    big = np.full(6, 2 ** 31 - 1, dtype=np.int32)
    xp, wp = np.full((1, 5, 3, 3), 127, dtype=np.int8), np.full((6, 5, 3, 3), 127, dtype=np.int8)
    with pytest.raises(OverflowError):
        oracle.conv2d_int8(xp, wp, 1, 0, 1, 0, bias=big)


@pytest.mark.parametrize("groups", [2, 3, 6])
def test_grouped_conv_is_block_diagonal_dense_conv(groups):
    """A grouped convolution is the dense convolution whose [K][C] filter matrix is block diagonal
    (zeros where output channel and input channel belong to different groups); groups = C = K is the
    depth-wise case.  Pins the group indexing against the dense path, which the other pins fix."""
    C, K = 6, 12 if groups != 6 else 6
    x = int8_uniform((2, C, 9, 7), 91)
    w = int8_uniform((K, C // groups, 3, 2), 92)
    Cg, Kg = C // groups, K // groups
    dense = np.zeros((K, C, 3, 2), dtype=np.int8)
    for k in range(K):
        g = k // Kg
        dense[k, g * Cg:(g + 1) * Cg] = w[k]
    bias = (int8_uniform((K,), 93).astype(np.int32) * 77)
    got = oracle.conv2d_int8(x, w, (2, 1), (1, 0), 1, 5, groups=groups, bias=bias, relu=True)
    want = oracle.conv2d_int8(x, dense, (2, 1), (1, 0), 1, 5, bias=bias, relu=True)
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1])
    # one group is the dense convolution; depth-wise with all-ones data counts the taps inside the image
    if groups == 6:
        ones = oracle.conv2d_int8(np.ones((1, 6, 4, 4), np.int8), np.ones((6, 1, 3, 3), np.int8), 1, 1, 1, 0, groups=6)[0]
        assert ones[0, :, 0, 0].tolist() == [4] * 6 and ones[0, :, 1, 1].tolist() == [9] * 6 and ones[0, :, 0, 2].tolist() == [6] * 6
