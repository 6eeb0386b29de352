"""Parity of the CUDA path against the CPU oracle, bit for bit, through the C ABI."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2104_04731_b200 as b2c
from paper_2104_04731_b200.synth import CONFIGS, int8_uniform

from gpu_util import check_against_oracle, run_embedding, to_dev

pytestmark = pytest.mark.gpu

_ref_cache = {}


def cfg_reference(cfg):
    if cfg.name not in _ref_cache:
        x, w = cfg.tensors()
        _ref_cache[cfg.name] = (x, w, oracle.conv2d_int8(x, w, cfg.stride, cfg.pad, cfg.dilation, cfg.shift))
    return _ref_cache[cfg.name]


# ---- layout kernels on their own ---------------------------------------------------------------------
@pytest.mark.parametrize("shape,C_pad", [((1, 16, 14, 14), 32), ((2, 3, 30, 23), 16), ((3, 70, 9, 13), 96),
                                         ((2, 256, 14, 14), 256), ((1, 1, 96, 480), 32), ((2, 64, 56, 56), 64),
                                         ((1500, 16, 14, 14), 32), ((1203, 48, 6, 10), 64)])   # large batches of small images
def test_pack_activations(lib, shape, C_pad):
    x = int8_uniform(shape, 301)
    want = oracle.pack_nhwc_cpad(x, C_pad)
    out = torch.full(want.shape, 55, dtype=torch.int8, device="cuda")
    lib.pack_activations(to_dev(x), out, C_pad)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), want)


@pytest.mark.parametrize("geom", [(2, 3, 20, 21, 7, 7, 2, 3, 1), (1, 1, 30, 60, 9, 21, 2, 0, 1), (2, 16, 9, 9, 3, 3, 1, 1, 1),
                                  (1, 5, 17, 13, 3, 2, (2, 1), (0, 2), (2, 3))])
@pytest.mark.parametrize("in_layout", [0, 1])
def test_im2col_matrix(lib, geom, in_layout):
    N, C, H, W, R, S, stride, pad, dil = geom
    x = int8_uniform((N, C, H, W), 302)
    A = oracle.im2col(x, R, S, stride, pad, dil)
    K_pad = -(-A.shape[1] // 32) * 32
    d = lib.make_desc(N, C, H, W, 1, R, S, stride, pad, dil, in_layout=in_layout)
    xin = x if in_layout == 0 else x.transpose(0, 2, 3, 1)
    out = torch.full((A.shape[0], K_pad), 55, dtype=torch.int8, device="cuda")
    lib.im2col(d, to_dev(xin), out, K_pad)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert np.array_equal(got[:, :A.shape[1]], A)
    assert not got[:, A.shape[1]:].any()


# ---- the five benchmark shapes, every enumerated embedding ------------------------------------------
@pytest.mark.parametrize("cfg", CONFIGS, ids=lambda c: c.name)
def test_config_every_embedding(lib, cfg):
    x, w, ref = cfg_reference(cfg)
    d = lib.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad, cfg.dilation, cfg.shift,
                      out_mode=cfg.out_mode)
    embs = lib.enumerate_embeddings(d)
    assert {0, 1, 2} <= {e.variant for e in embs}
    for e in embs:
        check_against_oracle(x, w, cfg.stride, cfg.pad, cfg.dilation, cfg.shift, cfg.out_mode, e.id, ref=ref)


@pytest.mark.parametrize("cfg", CONFIGS, ids=lambda c: c.name)
@pytest.mark.parametrize("in_layout,out_layout", [(1, 1), (0, 1), (1, 0)])
def test_config_layouts(lib, cfg, in_layout, out_layout):
    x, w, ref = cfg_reference(cfg)
    for variant in (0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10):
        d = lib.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad, cfg.dilation, cfg.shift,
                          in_layout, out_layout, 3)
        ids = [e.id for e in lib.enumerate_embeddings(d) if e.variant == variant]
        for i in ids[:2] + ids[-1:]:
            check_against_oracle(x, w, cfg.stride, cfg.pad, cfg.dilation, cfg.shift, 3, i, ref=ref,
                                 in_layout=in_layout, out_layout=out_layout)


# ---- randomised small shapes: ragged tiles, odd channels, strides, dilation, big pads, shifts -------
def _random_cases():
    rng = np.random.default_rng(2104)
    cases = []
    for i in range(36):
        C = int(rng.choice([1, 2, 3, 5, 17, 32, 33, 64, 72, 130]))
        K = int(rng.choice([1, 8, 15, 16, 17, 40, 64, 129]))
        R, S = int(rng.integers(1, 5)), int(rng.integers(1, 6))
        sh, sw = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        dh, dw = int(rng.integers(1, 4)), int(rng.integers(1, 3))
        ph, pw = int(rng.integers(0, 4)), int(rng.integers(0, 5))
        H = int(rng.integers(dh * (R - 1) + 1, dh * (R - 1) + 20))
        W = int(rng.integers(dw * (S - 1) + 1, dw * (S - 1) + 24))
        N = int(rng.integers(1, 4))
        shift = int(rng.choice([0, 1, 8, 12, 31]))
        cases.append((N, C, H, W, K, R, S, (sh, sw), (ph, pw), (dh, dw), shift, 400 + i))
    return cases


@pytest.mark.parametrize("case", _random_cases(), ids=lambda c: "n%dc%dh%dw%dk%dr%ds%d" % c[:7])
def test_random_shapes(lib, case):
    N, C, H, W, K, R, S, stride, pad, dil, shift, seed = case
    x = int8_uniform((N, C, H, W), seed)
    w = int8_uniform((K, C, R, S), seed + 1000)
    ref = oracle.conv2d_int8(x, w, stride, pad, dil, shift)
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, out_mode=3)
    embs = lib.enumerate_embeddings(d)
    for variant in (0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10):
        ids = [e.id for e in embs if e.variant == variant]
        for i in ids[:1] + ids[-1:]:
            check_against_oracle(x, w, stride, pad, dil, shift, 3, i, ref=ref)
    # NHWC in and out through the lowest-overhead embedding that accepts it
    d2 = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, 1, 1, 3)
    e2 = lib.enumerate_embeddings(d2)[0]
    check_against_oracle(x, w, stride, pad, dil, shift, 3, e2.id, ref=ref, in_layout=1, out_layout=1)


# ---- NHWC input whose channel count is no multiple of 32: re-padded into the scratch tensor -----------------
@pytest.mark.parametrize("C", [3, 24, 40, 72])
def test_nhwc_input_is_repadded_for_the_channel_pack_maps(lib, C):
    N, H, W, K, R, S = 3, 13, 15, 40, 3, 3
    x = int8_uniform((N, C, H, W), 771)
    w = int8_uniform((K, C, R, S), 772)
    ref = oracle.conv2d_int8(x, w, 1, 1, 1, 7)
    d = lib.make_desc(N, C, H, W, K, R, S, 1, 1, 1, 7, 1, 1, 3)
    embs = [e for e in lib.enumerate_embeddings(d) if e.variant in (b2c.VARIANT_CP_TMA, b2c.VARIANT_CP_SHIFT)]
    assert {e.variant for e in embs} == {b2c.VARIANT_CP_TMA, b2c.VARIANT_CP_SHIFT} and all(e.workspace_bytes > 0 for e in embs)
    seen = set()
    for e in embs:
        if (e.variant, e.tile_m) in seen:
            continue
        seen.add((e.variant, e.tile_m))
        check_against_oracle(x, w, 1, 1, 1, 7, 3, e.id, ref=ref, in_layout=1, out_layout=1)


# ---- swapped axis map (M <- k, N <- fused pixels) -------------------------------------------------------
@pytest.mark.parametrize("case", [
    # N, C, H, W, K, R, S, stride, pad, dil, shift
    (2, 32, 9, 11, 64, 3, 3, 1, 1, 1, 8),          # one channel tile half full
    (3, 40, 7, 7, 129, 3, 2, (2, 1), (1, 0), 1, 9),   # two channel tiles, the second with one row; images of 12 pixels
    (1, 256, 14, 14, 200, 3, 3, 2, 1, 1, 10),      # 49 pixels: runs cross no image boundary, ragged channel tile
    (5, 3, 20, 21, 96, 5, 5, 2, 2, (1, 2), 6),     # low channel count: row-unroll / space-to-depth / explicit views
    (2, 64, 30, 30, 128, 1, 1, 1, 0, 1, 7),        # 1x1, 1800 pixels: several 256-pixel tiles and a tail
])
@pytest.mark.parametrize("out_layout", [0, 1])
def test_swapped_axis_map(lib, case, out_layout):
    N, C, H, W, K, R, S, stride, pad, dil, shift = case
    x = int8_uniform((N, C, H, W), 611)
    w = int8_uniform((K, C, R, S), 612)
    ref = oracle.conv2d_int8(x, w, stride, pad, dil, shift)
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, 0, out_layout, 3)
    swapped = [e for e in lib.enumerate_embeddings(d) if e.map_m == b2c.AXIS_K]
    assert swapped and all(e.map_n == b2c.AXIS_NPQ and e.tile_m == 128 for e in swapped)
    seen = set()
    for e in swapped:
        key = (e.variant, e.tile_n, min(e.split_k, 2))
        if key in seen:
            continue
        seen.add(key)
        check_against_oracle(x, w, stride, pad, dil, shift, 3, e.id, ref=ref, out_layout=out_layout)
    # int8-only output through a split reduction goes through the scratch buffer and the finish kernel
    d8 = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, 0, out_layout, 2)
    split = [e for e in lib.enumerate_embeddings(d8) if e.map_m == b2c.AXIS_K and e.split_k > 1]
    if split:
        check_against_oracle(x, w, stride, pad, dil, shift, 2, split[0].id, ref=ref, out_layout=out_layout)


# ---- dilation phase pack (Image Pack of a dilated conv: phases fused into the batch) ---------------------
@pytest.mark.parametrize("case", [
    # N, C, H, W, K, R, S, pad, dil, shift
    (1, 16, 20, 20, 24, 3, 3, 2, 2, 8),             # "same" dilated 3x3, even image
    (2, 3, 17, 23, 16, 3, 3, (4, 4), (4, 4), 6),    # dilation 4, odd image: phase sub-images of unequal size
    (2, 5, 19, 14, 40, 3, 2, (1, 0), (2, 3), 7),    # pad not a multiple of the dilation; mixed dilation
    (1, 32, 13, 13, 8, 2, 4, (0, 5), (3, 1), 5),    # only the vertical axis dilated, wide horizontal padding
    (3, 64, 9, 31, 130, 3, 3, (3, 1), (3, 2), 9),   # several column tiles, ragged rows
])
@pytest.mark.parametrize("layouts", [(0, 0), (1, 1)])
def test_dilation_phase_pack(lib, case, layouts):
    N, C, H, W, K, R, S, pad, dil, shift = case
    in_layout, out_layout = layouts
    x = int8_uniform((N, C, H, W), 621)
    w = int8_uniform((K, C, R, S), 622)
    ref = oracle.conv2d_int8(x, w, 1, pad, dil, shift)
    d = lib.make_desc(N, C, H, W, K, R, S, 1, pad, dil, shift, in_layout, out_layout, 3)
    packs = [e for e in lib.enumerate_embeddings(d) if e.variant == b2c.VARIANT_DILATION_PACK]
    assert packs and all(e.map_k == b2c.AXIS_C and e.workspace_bytes > 0 for e in packs)
    seen = set()
    for e in packs:
        key = (e.tile_n, min(e.split_k, 2))
        if key in seen:
            continue
        seen.add(key)
        check_against_oracle(x, w, 1, pad, dil, shift, 3, e.id, ref=ref, in_layout=in_layout, out_layout=out_layout)
    # not listed without dilation or with a stride
    for (st, dl) in [(1, 1), (2, 2)]:
        d2 = lib.make_desc(N, C, H + 8, W + 8, K, R, S, st, pad, dl, shift)
        assert all(e.variant != b2c.VARIANT_DILATION_PACK for e in lib.enumerate_embeddings(d2))


def test_rewrite_and_convolve_halves(lib):
    # b2c_plan_rewrite_activations + b2c_conv2d_int8_run_rewritten = b2c_conv2d_int8_run, for every variant
    cfg = CONFIGS[0]
    x, w, ref = cfg_reference(cfg)
    x2 = int8_uniform(x.shape, 631)
    d = lib.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad, cfg.dilation, cfg.shift,
                      out_mode=3)
    seen = set()
    for e in lib.enumerate_embeddings(d):
        if e.variant in seen:
            continue
        seen.add(e.variant)
        plan = lib.Plan(d, e.id)
        data_b, weight_b = plan.footprint()
        assert weight_b >= w.size and (data_b > 0) == (e.variant in (0, 1, 4, 5, 7, 8, 9))
        assert data_b <= plan.workspace_bytes()
        ws = torch.zeros(max(16, plan.workspace_bytes()), dtype=torch.uint8, device="cuda")
        y32 = torch.zeros(ref[0].shape, dtype=torch.int32, device="cuda")
        y8 = torch.zeros(ref[1].shape, dtype=torch.int8, device="cuda")
        plan.set_weights(to_dev(w))
        plan.rewrite_activations(to_dev(x), ws)
        # a different tensor as x: variants with a rewrite must read the workspace, not x
        xin = to_dev(x2) if data_b else to_dev(x)
        plan.run_rewritten(xin, y32, y8, ws)
        torch.cuda.synchronize()
        assert plan.device_status() == b2c.OK
        assert np.array_equal(y32.cpu().numpy(), ref[0]) and np.array_equal(y8.cpu().numpy(), ref[1]), e.variant
        plan.destroy()


# ---- activation step (bias + ReLU) fused into every epilogue ---------------------------------------------
@pytest.mark.parametrize("case", [
    # N, C, H, W, K, R, S, stride, pad, dil, shift, out_mode
    (1, 16, 14, 14, 16, 3, 3, 1, 1, 1, 8, 3),      # small: every variant, split reductions through memory
    (2, 64, 12, 12, 136, 3, 3, 1, 1, 1, 9, 3),     # cluster reductions, swapped map, two channel tiles
    (1, 256, 7, 7, 64, 3, 3, 1, 1, 1, 10, 2),      # int8 only: split goes through the scratch and the finish kernel
    (2, 8, 20, 20, 24, 3, 3, 1, 2, 2, 6, 1),       # dilated (phase pack), int32 only: split meets in the output itself
])
@pytest.mark.parametrize("out_layout", [0, 1])
def test_bias_and_relu(lib, case, out_layout):
    N, C, H, W, K, R, S, stride, pad, dil, shift, out_mode = case
    x = int8_uniform((N, C, H, W), 641)
    w = int8_uniform((K, C, R, S), 642)
    bias = (int8_uniform((K,), 643).astype(np.int32) * 3001)
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, 0, out_layout, out_mode)
    P, Q = lib.out_shape(d)
    oshape = (N, K, P, Q) if out_layout == 0 else (N, P, Q, K)
    refs = {(b, r): oracle.conv2d_int8(x, w, stride, pad, dil, shift, bias=bias if b else None, relu=r)
            for b in (0, 1) for r in (False, True)}
    assert (refs[(1, False)][0] < 0).any()  # the ReLU has something to clip
    seen = set()
    xd, wd, bd = to_dev(x), to_dev(w), to_dev(bias)
    for e in lib.enumerate_embeddings(d):
        key = (e.variant, e.map_m, min(e.split_k, 2), e.tile_n >= 32 * e.split_k)
        if key in seen:
            continue
        seen.add(key)
        plan = lib.Plan(d, e.id)
        ws = torch.zeros(max(16, plan.workspace_bytes()), dtype=torch.uint8, device="cuda")
        plan.set_weights(wd)
        for (b, r) in [(1, True), (1, False), (0, True), (0, False)]:  # the last pair removes the step again
            plan.set_activation(bd if b else None, r)
            y32 = torch.full(oshape, -7777777, dtype=torch.int32, device="cuda") if out_mode & 1 else None
            y8 = torch.full(oshape, 77, dtype=torch.int8, device="cuda") if out_mode & 2 else None
            plan.run(xd, y32, y8, ws)
            torch.cuda.synchronize()
            tag = "variant %d map_m %d tile %d split %d bias %d relu %d" % (e.variant, e.map_m, e.tile_n, e.split_k, b, r)
            for got, want in ((y32, refs[(b, r)][0]), (y8, refs[(b, r)][1])):
                if got is None:
                    continue
                g = got.cpu().numpy()
                g = g if out_layout == 0 else g.transpose(0, 3, 1, 2)
                assert np.array_equal(g, want), tag
        assert plan.device_status() == b2c.OK
        plan.destroy()
    assert len(seen) >= 6


def test_chained_layers_skip_the_activation_pack(lib):
    # Layout coordination between layers: an int8 NHWC output with a multiple of 32 channels is the
    # channel-pack operand of the next layer as it stands, so the second plan has no rewrite at all.
    x = int8_uniform((2, 24, 18, 18), 651)
    w1 = int8_uniform((64, 24, 3, 3), 652)
    w2 = int8_uniform((40, 64, 3, 3), 653)
    bias1 = int8_uniform((64,), 654).astype(np.int32) * 500
    _, h_ref = oracle.conv2d_int8(x, w1, 1, 1, 1, 7, bias=bias1, relu=True)
    ref = oracle.conv2d_int8(h_ref, w2, 2, 1, 1, 9)
    d1 = lib.make_desc(2, 24, 18, 18, 64, 3, 3, 1, 1, 1, 7, b2c.LAYOUT_NCHW, b2c.LAYOUT_NHWC, b2c.OUT_I8)
    d2 = lib.make_desc(2, 64, 18, 18, 40, 3, 3, 2, 1, 1, 9, b2c.LAYOUT_NHWC, b2c.LAYOUT_NCHW, 3)
    p1 = lib.Plan(d1, b2c.POLICY_MIN_OVERHEAD)
    cp = [e for e in lib.enumerate_embeddings(d2) if e.variant == b2c.VARIANT_CP_TMA and e.split_k == 1]
    p2 = lib.Plan(d2, cp[0].id)
    assert p2.workspace_bytes() == 0 and p2.footprint()[0] == 0
    h = torch.zeros((2, 18, 18, 64), dtype=torch.int8, device="cuda")
    y32 = torch.zeros(ref[0].shape, dtype=torch.int32, device="cuda")
    y8 = torch.zeros(ref[1].shape, dtype=torch.int8, device="cuda")
    ws1 = torch.zeros(max(16, p1.workspace_bytes()), dtype=torch.uint8, device="cuda")
    p1.set_weights(to_dev(w1))
    p1.set_activation(to_dev(bias1), True)
    p2.set_weights(to_dev(w2))
    p1.run(to_dev(x), None, h, ws1)
    p2.run(h, y32, y8, None)
    torch.cuda.synchronize()
    assert np.array_equal(h.cpu().numpy().transpose(0, 3, 1, 2), h_ref)
    assert np.array_equal(y32.cpu().numpy(), ref[0]) and np.array_equal(y8.cpu().numpy(), ref[1])
    p1.destroy()
    p2.destroy()


@pytest.mark.parametrize("batch,cin,cout", [(1, 256, 512), (37, 72, 96), (300, 33, 17)])
def test_dense_layer_is_a_1x1_convolution(lib, batch, cin, cout):
    # A fully connected layer y = x W^T is the 1x1 convolution of a 1x1 image: M = batch, K = cout.
    x = int8_uniform((batch, cin, 1, 1), 661)
    w = int8_uniform((cout, cin, 1, 1), 662)
    want = x.reshape(batch, cin).astype(np.int64) @ w.reshape(cout, cin).astype(np.int64).T
    d = lib.make_desc(batch, cin, 1, 1, cout, 1, 1, out_mode=1)
    seen = set()
    for e in lib.enumerate_embeddings(d):
        if (e.variant, e.map_m) in seen:
            continue
        seen.add((e.variant, e.map_m))
        y32, _, _ = run_embedding(x, w, 1, 0, 1, 0, 1, e.id)
        assert np.array_equal(y32.reshape(batch, cout), want), (e.variant, e.map_m)


# ---- stencil as operand shift (stride-1 views: staged window, resident weights) -------------------------
@pytest.mark.parametrize("case", [
    # N, C, H, W, K, R, S, stride, pad, dil, shift
    (1, 16, 14, 14, 16, 3, 3, 1, 1, 1, 8),           # 32-byte channel block, padded width 16
    (2, 64, 20, 27, 64, 3, 3, 1, 1, 1, 9),           # 64-byte block, padded width 29 -> 32, tiles cross images
    (3, 128, 9, 9, 40, 3, 3, 1, 1, 1, 10),           # 128-byte block
    (1, 160, 11, 13, 24, 3, 2, 1, (2, 0), 1, 10),    # C_pad 160: five 32-byte blocks; asymmetric padding
    (2, 256, 8, 8, 16, 1, 1, 1, 0, 1, 9),            # 1x1: a single tap, two 128-byte blocks
    (2, 24, 19, 17, 48, 3, 3, 1, 2, 2, 7),           # dilated: shifts of two rows / two pixels
    (1, 8, 30, 250, 32, 5, 3, 1, (2, 1), 1, 6),      # wide rows (padded width 252 -> 256): windows of several rows
    (4, 3, 40, 40, 64, 7, 7, 2, 3, 1, 6),            # stride 2: only through space to depth
    (2, 1, 33, 61, 32, 9, 21, 2, 0, 1, 5),           # single channel, wide kernel, stride 2
    (2, 5, 21, 23, 20, 4, 5, (3, 2), (1, 2), 1, 5),  # stride 3 x 2
    (3, 2, 25, 27, 40, 5, 5, 2, 2, 1, 6),            # two channels, stride 2: three columns share a pixel (tap packing 3)
    (2, 1, 19, 40, 16, 3, 7, (1, 2), (1, 3), 1, 4),  # horizontal stride only: 2 phase bytes, tap packing 4 of S' = 4
])
@pytest.mark.parametrize("layouts", [(0, 0), (1, 1)])
def test_shift_execution(lib, case, layouts):
    N, C, H, W, K, R, S, stride, pad, dil, shift = case
    in_layout, out_layout = layouts
    x = int8_uniform((N, C, H, W), 671)
    w = int8_uniform((K, C, R, S), 672)
    ref = oracle.conv2d_int8(x, w, stride, pad, dil, shift)
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, in_layout, out_layout, 3)
    shifts = [e for e in lib.enumerate_embeddings(d) if e.variant in (b2c.VARIANT_CP_SHIFT, b2c.VARIANT_S2D_SHIFT)]
    want = {b2c.VARIANT_S2D_SHIFT} if stride != 1 else {b2c.VARIANT_CP_SHIFT}
    assert {e.variant for e in shifts} == want   # (an NHWC source without padded channels is re-padded into the scratch tensor)
    for e in shifts:
        assert e.split_k == 1 and e.tile_n >= K and e.map_m == b2c.AXIS_NPQ
        check_against_oracle(x, w, stride, pad, dil, shift, 3, e.id, ref=ref, in_layout=in_layout, out_layout=out_layout)


@pytest.mark.parametrize("case", [
    # N, C, H, W, K, R, S, stride, pad, dil, shift
    (4, 3, 40, 48, 64, 7, 7, 2, 3, 1, 6),              # the low-channel 7x7 stride-2 class: (dh, s, c) = 42 -> 64 channels
    (2, 1, 33, 64, 32, 9, 21, 2, 0, 1, 5),             # single channel, wide kernel: 42 -> 64, five filter rows left
    (2, 1, 30, 61, 32, 9, 21, (2, 2), (1, 3), 1, 5),   # rows not a multiple of 16 bytes: byte staging
    (3, 5, 21, 23, 20, 4, 5, (3, 2), (1, 2), (1, 2), 5),   # stride 3 x 2, horizontal dilation 2, ragged tiles
    (1, 16, 14, 14, 16, 3, 3, 1, 1, 1, 8),             # stride 1: plain row unroll, 48 -> 64 channels
    (2, 40, 12, 12, 24, 3, 3, (2, 1), 1, 1, 8),        # 2 * 3 * 40 = 240 -> 256 channels: two 128-byte blocks
    (1, 2, 70, 9, 8, 5, 2, (1, 1), (2, 0), 1, 4),      # tall image: many tile rows, one tile column
])
@pytest.mark.parametrize("layouts", [(0, 0), (1, 1)])
def test_row_phase_unroll_shift(lib, case, layouts):
    N, C, H, W, K, R, S, stride, pad, dil, shift = case
    in_layout, out_layout = layouts
    x = int8_uniform((N, C, H, W), 681)
    w = int8_uniform((K, C, R, S), 682)
    ref = oracle.conv2d_int8(x, w, stride, pad, dil, shift)
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, in_layout, out_layout, 3)
    es = [e for e in lib.enumerate_embeddings(d) if e.variant == b2c.VARIANT_ROWPHASE_SHIFT]
    assert len(es) == 1 and es[0].map_k == b2c.AXIS_SC and es[0].split_k == 1 and es[0].workspace_bytes > 0
    check_against_oracle(x, w, stride, pad, dil, shift, 3, es[0].id, ref=ref, in_layout=in_layout, out_layout=out_layout)
    # vertical dilation is outside this rewrite
    d2 = lib.make_desc(N, C, H + 8, W, K, R, S, stride, pad, (2, 1), shift)
    assert all(e.variant != b2c.VARIANT_ROWPHASE_SHIFT for e in lib.enumerate_embeddings(d2))


def test_shift_execution_long_tile_walk(lib):
    # about twelve tiles per block of the persistent grid: the window ring and both accumulator
    # buffers wrap several times (cfg 1's layer at batch 1800)
    x = int8_uniform((1800, 16, 14, 14), 675)
    w = int8_uniform((16, 16, 3, 3), 676)
    ref = oracle.conv2d_int8(x, w, 1, 1, 1, 8)
    d = lib.make_desc(1800, 16, 14, 14, 16, 3, 3, 1, 1, 1, 8, out_mode=3)
    e = next(e for e in lib.enumerate_embeddings(d) if e.variant == b2c.VARIANT_CP_SHIFT)
    check_against_oracle(x, w, 1, 1, 1, 8, 3, e.id, ref=ref)


def test_shift_execution_many_tiles(lib):
    # enough tiles (2800) for every block of the persistent grid to walk several: both accumulator buffers
    # wrap, and the two epilogue warps of each lane quadrant take alternate tiles (32 columns each)
    x = int8_uniform((400, 32, 28, 28), 673)
    w = int8_uniform((32, 32, 3, 3), 674)
    ref = oracle.conv2d_int8(x, w, 1, 1, 1, 9)
    d = lib.make_desc(400, 32, 28, 28, 32, 3, 3, 1, 1, 1, 9, out_mode=3)
    e = next(e for e in lib.enumerate_embeddings(d) if e.variant == b2c.VARIANT_CP_SHIFT)
    check_against_oracle(x, w, 1, 1, 1, 9, 3, e.id, ref=ref)


def test_shift_execution_four_accumulator_buffers(lib):
    # 64-column tiles use a ring of four accumulator buffers; cfg 2's layer at batch 120 gives every block
    # about eleven tiles, so the ring wraps more than twice (odd tile counts per block included)
    x = int8_uniform((120, 64, 56, 56), 677)
    w = int8_uniform((64, 64, 3, 3), 678)
    ref = oracle.conv2d_int8(x, w, 1, 1, 1, 10)
    d = lib.make_desc(120, 64, 56, 56, 64, 3, 3, 1, 1, 1, 10, out_mode=3)
    e = next(e for e in lib.enumerate_embeddings(d) if e.variant == b2c.VARIANT_CP_SHIFT)
    check_against_oracle(x, w, 1, 1, 1, 10, 3, e.id, ref=ref)


# ---- grouped / depth-wise convolution: one launch, the group is a grid axis of the kernel ------------------
@pytest.mark.parametrize("case", [
    # N, C, H, W, K, groups, R, S, stride, pad, dil, shift, out_mode
    (2, 8, 12, 16, 12, 2, 3, 3, 1, 1, 1, 6, 3),         # two groups of 4 -> 6 channels, rows of 16 bytes
    (3, 12, 9, 7, 24, 4, 3, 2, (2, 1), (1, 0), 1, 5, 3),  # four groups, odd image: unaligned channel slices
    (2, 6, 10, 10, 6, 6, 3, 3, 1, 1, 1, 4, 1),          # depth-wise, int32 only
    (1, 16, 20, 20, 16, 16, 5, 5, 2, 2, 1, 5, 2),       # depth-wise 5x5 stride 2, int8 only
    (2, 64, 7, 7, 128, 2, 1, 1, 1, 0, 1, 7, 3),         # pointwise, 64 output channels per group
    (2, 256, 14, 14, 256, 256, 3, 3, 1, 1, 1, 4, 3),    # depth-wise, 256 channels: 256 groups in one launch
    (40, 32, 28, 28, 64, 8, 3, 3, 2, 1, 1, 6, 3),       # many tiles per group: the persistent walk with a group axis
    (2, 48, 9, 9, 96, 48, 3, 3, 1, 1, 1, 5, 3),         # 48 groups of 1 -> 2 channels: merged 16 at a time, three merged groups
])
def test_grouped_convolution(lib, case):
    N, C, H, W, K, groups, R, S, stride, pad, dil, shift, out_mode = case
    x = int8_uniform((N, C, H, W), 691)
    w = int8_uniform((K, C // groups, R, S), 692)
    bias = int8_uniform((K,), 693).astype(np.int32) * 211
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, out_mode=out_mode)
    P, Q = lib.out_shape(d)
    plan = lib.Plan(d, groups=groups)
    assert plan.workspace_bytes() == 0 and plan.info().variant in (b2c.VARIANT_IM2COL_GATHER, b2c.VARIANT_IM2COL_STAGED)
    xd, wd = to_dev(x), to_dev(w)
    plan.set_weights(wd)
    for use_bias, relu in [(False, False), (True, True)]:
        ref = oracle.conv2d_int8(x, w, stride, pad, dil, shift, groups=groups, bias=bias if use_bias else None, relu=relu)
        plan.set_activation(to_dev(bias) if use_bias else None, relu)
        y32 = torch.full((N, K, P, Q), -7777777, dtype=torch.int32, device="cuda") if out_mode & 1 else None
        y8 = torch.full((N, K, P, Q), 77, dtype=torch.int8, device="cuda") if out_mode & 2 else None
        plan.run(xd, y32, y8, None)
        torch.cuda.synchronize()
        assert plan.device_status() == b2c.OK
        if y32 is not None:
            assert np.array_equal(y32.cpu().numpy(), ref[0])
        if y8 is not None:
            assert np.array_equal(y8.cpu().numpy(), ref[1])
    plan.destroy()
    # argument checks: groups must divide both channel counts; whole tensors must be NCHW / NKPQ
    raw = lib.load()
    h = ctypes.c_void_p()
    assert raw.b2c_plan_create_grouped(ctypes.byref(d), 5, ctypes.byref(h)) == b2c.E_INVALID_ARG
    d_nhwc = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, 1, 0, out_mode)
    assert raw.b2c_plan_create_grouped(ctypes.byref(d_nhwc), groups, ctypes.byref(h)) == b2c.E_UNSUPPORTED


@pytest.mark.parametrize("case", [
    (2, 256, 14, 14, 256, 256, 3, 3, 1, 1, 1, 4, 3),    # depth-wise, 256 channels: the full merge wins on this device
    (3, 12, 9, 7, 24, 4, 3, 2, (2, 1), (1, 0), 1, 5, 3),  # four groups, odd image
    (2, 64, 7, 7, 128, 2, 1, 1, 1, 0, 1, 7, 2),         # pointwise, two wide groups
])
def test_grouped_convolution_form_chosen_by_timing(lib, case):
    N, C, H, W, K, groups, R, S, stride, pad, dil, shift, out_mode = case
    x = int8_uniform((N, C, H, W), 695)
    w = int8_uniform((K, C // groups, R, S), 696)
    bias = int8_uniform((K,), 697).astype(np.int32) * 101
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, out_mode=out_mode)
    P, Q = lib.out_shape(d)
    plan = lib.Plan(d, b2c.POLICY_AUTO_TIMED, groups=groups)
    assert plan.info().device_us > 0
    ws = torch.empty(max(16, plan.workspace_bytes()), dtype=torch.uint8, device="cuda")
    plan.set_weights(to_dev(w))
    xd = to_dev(x)
    for use_bias, relu in [(False, False), (True, True)]:
        ref = oracle.conv2d_int8(x, w, stride, pad, dil, shift, groups=groups, bias=bias if use_bias else None, relu=relu)
        plan.set_activation(to_dev(bias) if use_bias else None, relu)
        y32 = torch.full((N, K, P, Q), -7777777, dtype=torch.int32, device="cuda") if out_mode & 1 else None
        y8 = torch.full((N, K, P, Q), 77, dtype=torch.int8, device="cuda") if out_mode & 2 else None
        plan.run(xd, y32, y8, ws)
        torch.cuda.synchronize()
        assert plan.device_status() == b2c.OK
        if y32 is not None:
            assert np.array_equal(y32.cpu().numpy(), ref[0])
        if y8 is not None:
            assert np.array_equal(y8.cpu().numpy(), ref[1])
    plan.destroy()


def test_extreme_values_and_shift_clip(lib):
    # -128 * -128 is the largest product; all-(-128) tensors with 9*64 taps reach 9437184.
    x = np.full((1, 64, 6, 6), -128, dtype=np.int8)
    w = np.full((16, 64, 3, 3), -128, dtype=np.int8)
    ref = oracle.conv2d_int8(x, w, 1, 1, 1, 16)
    for variant in (0, 1, 2, 3, 4, 5, 6, 7, 8, 9):
        d = lib.make_desc(1, 64, 6, 6, 16, 3, 3, 1, 1, 1, 16, out_mode=3)
        ids = [e.id for e in lib.enumerate_embeddings(d) if e.variant == variant]
        if ids:
            check_against_oracle(x, w, 1, 1, 1, 16, 3, ids[0], ref=ref)
    x = int8_uniform((1, 32, 5, 5), 501)
    w = int8_uniform((8, 32, 3, 3), 502)
    for shift in (0, 1, 8, 31):
        ref = oracle.conv2d_int8(x, w, 1, 1, 1, shift)
        check_against_oracle(x, w, 1, 1, 1, shift, 2, b2c.POLICY_MIN_OVERHEAD, ref=ref)


# ---- the other entry points -----------------------------------------------------------------------------
def test_one_shot_device_and_host_calls(lib):
    for cfg in (CONFIGS[0], CONFIGS[3]):
        x, w, ref = cfg_reference(cfg)
        xd, wd = to_dev(x), to_dev(w)
        y32 = torch.zeros(ref[0].shape, dtype=torch.int32, device="cuda")
        y8 = torch.zeros(ref[0].shape, dtype=torch.int8, device="cuda")
        for _ in range(2):  # the second call reuses the cached plan
            lib.conv2d_int8(xd, wd, cfg.stride, cfg.pad, cfg.dilation, cfg.shift, y32, y8)
            torch.cuda.synchronize()
            assert np.array_equal(y32.cpu().numpy(), ref[0])
            assert np.array_equal(y8.cpu().numpy(), ref[1])
        h32 = np.zeros(ref[0].shape, dtype=np.int32)
        h8 = np.zeros(ref[0].shape, dtype=np.int8)
        lib.conv2d_int8_host(x, w, cfg.stride, cfg.pad, cfg.dilation, cfg.shift, h32, h8)
        assert np.array_equal(h32, ref[0]) and np.array_equal(h8, ref[1])
        h8[:] = 0
        lib.conv2d_int8_host(x, w, cfg.stride, cfg.pad, cfg.dilation, cfg.shift, None, h8)
        assert np.array_equal(h8, ref[1])


def test_policies(lib):
    cfg = CONFIGS[0]
    x, w, ref = cfg_reference(cfg)
    for policy in (b2c.POLICY_AUTO_TIMED, b2c.POLICY_AUTO_TIMED_CONCURRENT, b2c.POLICY_MIN_OVERHEAD,
                   b2c.POLICY_MIN_WORKSPACE):
        emb = check_against_oracle(x, w, cfg.stride, cfg.pad, cfg.dilation, cfg.shift, cfg.out_mode, policy, ref=ref)
        if policy in (b2c.POLICY_AUTO_TIMED, b2c.POLICY_AUTO_TIMED_CONCURRENT):
            assert emb.device_us > 0
        if policy == b2c.POLICY_MIN_WORKSPACE:
            assert emb.workspace_bytes == 0


def test_error_paths_on_device(lib):
    cfg = CONFIGS[0]
    d = lib.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad, out_mode=3)
    raw = lib.load()
    plan = lib.Plan(d, b2c.POLICY_MIN_OVERHEAD)
    x, w = (to_dev(t) for t in cfg.tensors())
    y32 = torch.zeros((1, 16, 14, 14), dtype=torch.int32, device="cuda")
    y8 = torch.zeros((1, 16, 14, 14), dtype=torch.int8, device="cuda")
    ws = torch.zeros(max(16, plan.workspace_bytes()), dtype=torch.uint8, device="cuda")
    p = lambda t: ctypes.c_void_p(t.data_ptr()) if t is not None else None
    assert raw.b2c_conv2d_int8_run(plan._h, p(x), p(y32), p(y8), p(ws), None) == b2c.E_NOT_READY
    plan.set_weights(w)
    assert raw.b2c_conv2d_int8_run(plan._h, p(x), None, p(y8), p(ws), None) == b2c.E_INVALID_ARG
    assert raw.b2c_conv2d_int8_run(plan._h, p(x), p(y32), None, p(ws), None) == b2c.E_INVALID_ARG
    assert raw.b2c_conv2d_int8_run(plan._h, ctypes.c_void_p(x.data_ptr() + 1), p(y32), p(y8), p(ws), None) == b2c.E_INVALID_ARG
    h = ctypes.c_void_p()
    assert raw.b2c_plan_create(ctypes.byref(d), 10 ** 6, None, ctypes.byref(h)) == b2c.E_INVALID_ARG
    assert raw.b2c_plan_create(ctypes.byref(d), -9, None, ctypes.byref(h)) == b2c.E_INVALID_ARG
    plan.run(x, y32, y8, ws)
    torch.cuda.synchronize()
    assert plan.device_status() == b2c.OK
    plan.destroy()


# ---- kernels of consecutive calls overlap their launch and set-up; memory effects must stay in stream order ----
@pytest.mark.parametrize("variant", [0, 1, 2, 3, 4])
def test_back_to_back_runs_keep_stream_order(lib, variant):
    cfg = CONFIGS[0]
    xa, w = cfg.tensors(0)
    xb, _ = cfg.tensors(1)
    refs = [oracle.conv2d_int8(x, w, cfg.stride, cfg.pad, cfg.dilation, cfg.shift) for x in (xa, xb)]
    d = lib.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad, cfg.dilation, cfg.shift,
                      out_mode=3)
    eid = next(e.id for e in lib.enumerate_embeddings(d) if e.variant == variant and e.split_k == 1)
    plan = lib.Plan(d, eid)
    xs = [to_dev(xa), to_dev(xb)]
    plan.set_weights(to_dev(w))
    ws = torch.zeros(max(16, plan.workspace_bytes()), dtype=torch.uint8, device="cuda")  # shared by all calls
    outs = [(torch.zeros(refs[0][0].shape, dtype=torch.int32, device="cuda"),
             torch.zeros(refs[0][0].shape, dtype=torch.int8, device="cuda")) for _ in range(40)]

    def enqueue():
        for i, (y32, y8) in enumerate(outs):
            plan.run(xs[i & 1], y32, y8, ws)

    enqueue()
    torch.cuda.synchronize()
    for i, (y32, y8) in enumerate(outs):
        assert np.array_equal(y32.cpu().numpy(), refs[i & 1][0]), i
        assert np.array_equal(y8.cpu().numpy(), refs[i & 1][1]), i
        y32.zero_()
        y8.zero_()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        enqueue()
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    for i, (y32, y8) in enumerate(outs):
        assert np.array_equal(y32.cpu().numpy(), refs[i & 1][0]), i
        assert np.array_equal(y8.cpu().numpy(), refs[i & 1][1]), i
    assert plan.device_status() == b2c.OK
    plan.destroy()


# ---- grids much larger than the machine: persistent blocks, two accumulator buffers --------------------
@pytest.mark.parametrize("tile_n", [32, 128])
def test_large_grid_persistent_tiles(lib, tile_n):
    N, C, H, W, K, R, S = 56, 64, 28, 28, 128, 3, 3   # 43904 output pixels = 343 row tiles (> 2 per SM)
    x = int8_uniform((N, C, H, W), 701)
    w = int8_uniform((K, C, R, S), 702)
    ref = oracle.conv2d_int8(x, w, 1, 1, 1, 9)
    for in_layout, out_layout in ((0, 0), (1, 1)):
        d = lib.make_desc(N, C, H, W, K, R, S, 1, 1, 1, 9, in_layout, out_layout, 3)
        for variant in (0, 1):
            ids = [e.id for e in lib.enumerate_embeddings(d) if e.variant == variant and e.tile_n == tile_n and e.split_k == 1]
            assert ids
            check_against_oracle(x, w, 1, 1, 1, 9, 3, ids[0], ref=ref, in_layout=in_layout, out_layout=out_layout)


# ---- the wide persistent schedule the large-batch benchmark runs: 128 x 256 tiles, two 256-column
# accumulators (all of tensor memory), one block per SM walking 614 tiles -------------------------------
_wide_ref = {}


@pytest.mark.parametrize("in_layout", [0, 1])
@pytest.mark.parametrize("out_mode", [1, 2, 3])
def test_persistent_256_column_tiles(lib, in_layout, out_mode):
    N, C, H, W, K, R, S = 800, 64, 14, 14, 512, 3, 3   # stride 2, pad 1: 39200 pixels = 307 row tiles x 2 column tiles
    if "ref" not in _wide_ref:
        x = int8_uniform((N, C, H, W), 711)
        w = int8_uniform((K, C, R, S), 712)
        _wide_ref["ref"] = (x, w, oracle.conv2d_int8(x, w, 2, 1, 1, 10))
    x, w, ref = _wide_ref["ref"]
    d = lib.make_desc(N, C, H, W, K, R, S, 2, 1, 1, 10, in_layout, 0, out_mode)
    ids = [e.id for e in lib.enumerate_embeddings(d) if e.variant == 0 and e.tile_n == 256 and e.split_k == 1
           and e.map_m == b2c.AXIS_NPQ]
    assert ids
    check_against_oracle(x, w, 2, 1, 1, 10, out_mode, ids[0], ref=ref, in_layout=in_layout)


# ---- two-SM schedule: a pair of blocks per 256-row tile, each loading half of the column tile -------------
@pytest.mark.parametrize("case", [
    # N, C, H, W, K, R, S, stride, pad, dil, shift
    (32, 256, 14, 14, 512, 3, 3, 2, 1, 1, 10),     # the compute-bound benchmark shape: 7 x 2 pair tiles, the last one half empty
    (3, 64, 20, 20, 129, 3, 3, 1, 1, 1, 9),        # ragged column tile (129 channels), 1200 pixels
    (2, 32, 17, 13, 40, 2, 3, (1, 2), (0, 1), (2, 1), 7),   # 8-row-group ragged weights, dilation, odd pixel count
    (5, 3, 30, 31, 96, 5, 5, 2, 2, 1, 6),          # low channel count: row-unroll / space-to-depth / explicit views
    (1, 16, 33, 33, 64, 3, 3, 1, 2, 2, 8),         # dilated: the phase pack's scattered rows
    (1, 128, 12, 11, 256, 1, 1, 1, 0, 1, 5),       # 1x1: 132 pixels, the second block of the pair nearly empty
])
@pytest.mark.parametrize("out_layout", [0, 1])
def test_two_sm_schedule(lib, case, out_layout):
    N, C, H, W, K, R, S, stride, pad, dil, shift = case
    x = int8_uniform((N, C, H, W), 731)
    w = int8_uniform((K, C, R, S), 732)
    ref = oracle.conv2d_int8(x, w, stride, pad, dil, shift)
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, 0, out_layout, 3)
    pairs = [e for e in lib.enumerate_embeddings(d) if e.tile_m == 256]
    assert pairs and all(e.split_k == 1 and e.map_m == b2c.AXIS_NPQ and e.tile_n >= 32 for e in pairs)
    for e in pairs:
        check_against_oracle(x, w, stride, pad, dil, shift, 3, e.id, ref=ref, out_layout=out_layout)


@pytest.mark.parametrize("in_layout", [0, 1])
@pytest.mark.parametrize("tile_n", [64, 256])
def test_two_sm_schedule_walks_tiles(lib, in_layout, tile_n):
    """More pair tiles than SM pairs: the clusters walk the tile list with two accumulator buffers."""
    N, C, H, W, K, R, S = 800, 64, 14, 14, 512, 3, 3   # 39200 pixels = 154 pair row tiles x 2 (or 8) column tiles
    if "ref" not in _wide_ref:
        x = int8_uniform((N, C, H, W), 711)
        w = int8_uniform((K, C, R, S), 712)
        _wide_ref["ref"] = (x, w, oracle.conv2d_int8(x, w, 2, 1, 1, 10))
    x, w, ref = _wide_ref["ref"]
    d = lib.make_desc(N, C, H, W, K, R, S, 2, 1, 1, 10, in_layout, 0, 3)
    for variant in (0, 1):
        ids = [e.id for e in lib.enumerate_embeddings(d) if e.variant == variant and e.tile_n == tile_n and e.tile_m == 256]
        assert ids
        check_against_oracle(x, w, 2, 1, 1, 10, 3, ids[0], ref=ref, in_layout=in_layout)


# ---- stencil unroll from a TMA-staged two-dimensional window (low-channel shapes, NCHW rows of 16-byte multiples) ---
@pytest.mark.parametrize("case", [
    # N, C, H, W, K, R, S, stride, pad, dil, shift
    (2, 3, 40, 48, 64, 7, 7, 2, 3, 1, 6),              # the 7x7 stride-2 stem class
    (3, 1, 30, 96, 32, 9, 21, 2, 0, 1, 5),             # single channel, wide kernel: runs of 24 straddle 16-byte chunks
    (2, 2, 17, 32, 17, 3, 3, 1, 1, 1, 4),              # 17 output channels in a 32-column tile, odd height
    (1, 5, 33, 64, 130, 5, 4, (3, 1), (2, 3), (2, 1), 7),  # vertical dilation, stride 3 x 1, 130 channels (256-column tile)
    (4, 1, 9, 16, 8, 3, 5, (1, 2), (1, 2), 1, 3),      # narrow image: 16-pixel-wide tiles
    (2, 4, 20, 240, 40, 1, 1, 1, 0, 1, 2),             # 1x1 kernel: runs of one tap padded to four
    (1, 16, 12, 16, 16, 3, 3, 1, 1, 1, 8),             # 16 channels: 576-byte rows, five reduction blocks
    # small images: linear tiles over whole images, border taps masked
    (5, 16, 14, 14, 16, 3, 3, 1, 1, 1, 8),             # the 14 x 14, 16-channel shape: tiles span two images
    (7, 2, 10, 8, 40, 3, 5, 2, 2, (2, 1), 5),          # stride 2, pad 2, vertical dilation; 20 pixels... too few: not listed
    (9, 2, 20, 24, 33, 3, 5, (2, 1), (2, 1), (2, 1), 5),   # runs of two words, vertical dilation, 240 pixels per image
    (3, 4, 9, 12, 8, 1, 1, 1, (1, 3), 1, 2),           # 1x1 kernel with padding: outputs that see only zeros
    (6, 1, 16, 16, 64, 5, 8, (1, 2), (2, 4), 1, 6),    # 16-byte rows but small: the linear form is preferred; 8-tap runs
])
@pytest.mark.parametrize("out_layout,out_mode", [(0, 3), (1, 3), (0, 2)])
def test_tma_window_unroll(lib, case, out_layout, out_mode):
    N, C, H, W, K, R, S, stride, pad, dil, shift = case
    x = int8_uniform((N, C, H, W), 761)
    w = int8_uniform((K, C, R, S), 762)
    ref = oracle.conv2d_int8(x, w, stride, pad, dil, shift)
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, 0, out_layout, out_mode)
    ids = [e.id for e in lib.enumerate_embeddings(d) if e.variant == b2c.VARIANT_IM2COL_WINDOW]
    P, Q = lib.out_shape(d)
    if W % 16 != 0 and P * Q < 43:
        assert not ids   # neither form applies: rows are no 16-byte multiples and a tile would span too many images
        return
    assert len(ids) == 1
    check_against_oracle(x, w, stride, pad, dil, shift, out_mode, ids[0], ref=ref, out_layout=out_layout)


def test_window_unroll_small_images_walks_tiles(lib):
    """Linear tiles over many small images: the rings wrap, tiles start inside one image and end in the next."""
    N, C, H, W, K, R, S = 700, 16, 14, 14, 16, 3, 3   # 137200 pixels = 1072 tiles
    x = int8_uniform((N, C, H, W), 766)
    w = int8_uniform((K, C, R, S), 767)
    ref = oracle.conv2d_int8(x, w, 1, 1, 1, 8)
    d = lib.make_desc(N, C, H, W, K, R, S, 1, 1, 1, 8, 0, 0, 3)
    e = [e for e in lib.enumerate_embeddings(d) if e.variant == b2c.VARIANT_IM2COL_WINDOW][0]
    check_against_oracle(x, w, 1, 1, 1, 8, 3, e.id, ref=ref)


def test_tma_window_unroll_walks_tiles(lib):
    """More tiles than resident blocks (2 x 148): the rings of windows, operand buffers and accumulators wrap."""
    N, C, H, W, K, R, S = 12, 3, 112, 112, 64, 7, 7   # stride 2: 56 x 56 outputs, 28 x 1 tiles per image... 336 tiles
    x = int8_uniform((N, C, H, W), 763)
    w = int8_uniform((K, C, R, S), 764)
    bias = (int8_uniform((K,), 765).astype(np.int32) * 500)
    ref = oracle.conv2d_int8(x, w, 2, 3, 1, 7, bias=bias, relu=True)
    d = lib.make_desc(N, C, H, W, K, R, S, 2, 3, 1, 7, 0, 0, 3)
    e = [e for e in lib.enumerate_embeddings(d) if e.variant == b2c.VARIANT_IM2COL_WINDOW][0]
    plan = lib.Plan(d, e.id)
    plan.set_weights(to_dev(w))
    plan.set_activation(to_dev(bias), True)
    y32 = torch.full(ref[0].shape, -7777777, dtype=torch.int32, device="cuda")
    y8 = torch.full(ref[1].shape, 77, dtype=torch.int8, device="cuda")
    xd = to_dev(x)
    for _ in range(2):
        plan.run(xd, y32, y8, None)
    torch.cuda.synchronize()
    assert plan.device_status() == b2c.OK and plan.workspace_bytes() == 0
    assert np.array_equal(y32.cpu().numpy(), ref[0]) and np.array_equal(y8.cpu().numpy(), ref[1])
    plan.destroy()


# ---- activation pack inside the two-SM kernel (NCHW input, persistent channel-pack schedule) -------------
@pytest.mark.parametrize("case", [
    # N, C, H, W, K, R, S, stride, pad, shift, tile_n
    (100, 16, 14, 14, 64, 3, 3, 1, 1, 8, 64),     # whole image per unit, channels padded 16 -> 32
    (8, 64, 56, 56, 64, 3, 3, 1, 1, 9, 64),       # units of 256 pixels (rows of 3136 pixels), ragged last unit
    (60, 48, 20, 20, 96, 3, 3, 1, 1, 9, 32),      # 48 channels in 64-channel units: the last 16 are zero padding
    (450, 32, 7, 9, 40, 2, 2, 1, 0, 7, 64),       # HW = 63 is no multiple of 4: falls back to the separate pack kernel
])
def test_fused_activation_pack(lib, case):
    N, C, H, W, K, R, S, stride, pad, shift, tile_n = case
    x = int8_uniform((N, C, H, W), 751)
    w = int8_uniform((K, C, R, S), 752)
    bias = (int8_uniform((K,), 753).astype(np.int32) * 1000)
    ref = oracle.conv2d_int8(x, w, stride, pad, 1, shift, bias=bias, relu=True)
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, 1, shift, 0, 0, 3)
    ids = [e.id for e in lib.enumerate_embeddings(d) if e.variant == 0 and e.tile_m == 256 and e.tile_n == tile_n]
    assert ids
    plan = lib.Plan(d, ids[0])
    plan.set_weights(to_dev(w))
    plan.set_activation(to_dev(bias), True)
    y32 = torch.full(ref[0].shape, -7777777, dtype=torch.int32, device="cuda")
    y8 = torch.full(ref[1].shape, 77, dtype=torch.int8, device="cuda")
    ws = torch.empty(max(16, plan.workspace_bytes()), dtype=torch.uint8, device="cuda")
    ws.fill_(0xAB)
    xd = to_dev(x)
    for _ in range(2):   # twice: the counters in the workspace are cleared by every run
        plan.run(xd, y32, y8, ws)
    torch.cuda.synchronize()
    assert plan.device_status() == b2c.OK
    assert np.array_equal(y32.cpu().numpy(), ref[0]) and np.array_equal(y8.cpu().numpy(), ref[1])
    # the rewritten operand the kernel left in the workspace is the oracle's NHWC, channel-padded tensor
    C_pad = -(-C // 32) * 32
    want = oracle.pack_nhwc_cpad(x, C_pad)
    got = ws[:want.size].cpu().numpy().view(np.int8).reshape(want.shape)
    assert np.array_equal(got, want)
    g = torch.cuda.CUDAGraph()   # and once more from a captured graph, replayed twice
    y32.fill_(-1)
    with torch.cuda.graph(g):
        plan.run(xd, y32, y8, ws)
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    assert plan.device_status() == b2c.OK
    assert np.array_equal(y32.cpu().numpy(), ref[0]) and np.array_equal(y8.cpu().numpy(), ref[1])
    plan.destroy()


# ---- one-shot calls of one shape on two streams with different weights do not disturb each other ---------
def test_one_shot_calls_on_two_streams(lib):
    N, C, H, W, K, R, S = 2, 32, 20, 20, 48, 3, 3
    x = int8_uniform((N, C, H, W), 721)
    ws = [int8_uniform((K, C, R, S), 722 + i) for i in range(2)]
    refs = [oracle.conv2d_int8(x, w, 1, 1, 1, 7) for w in ws]
    xd = to_dev(x)
    wd = [to_dev(w) for w in ws]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [[(torch.zeros(refs[0][0].shape, dtype=torch.int32, device="cuda"),
              torch.zeros(refs[0][1].shape, dtype=torch.int8, device="cuda")) for _ in range(6)] for _ in range(2)]
    torch.cuda.synchronize()
    for rep in range(6):          # interleaved, nothing orders the two streams against each other
        for i in range(2):
            y32, y8 = outs[i][rep]
            lib.conv2d_int8(xd, wd[i], 1, 1, 1, 7, y32, y8, stream=streams[i])
    torch.cuda.synchronize()
    assert lib.oneshot_status() == b2c.OK
    for i in range(2):
        for y32, y8 in outs[i]:
            assert np.array_equal(y32.cpu().numpy(), refs[i][0])
            assert np.array_equal(y8.cpu().numpy(), refs[i][1])
    lib.oneshot_cache_clear()
    y32, y8 = outs[0][0]
    y32.zero_()
    lib.conv2d_int8(xd, wd[1], 1, 1, 1, 7, y32, y8)   # selects again after the cache was cleared
    torch.cuda.synchronize()
    assert np.array_equal(y32.cpu().numpy(), refs[1][0])


# ---- host-side fault injection: a tensor map the driver refuses ---------------------------------------
def test_failed_descriptor_encode_is_reported_and_skipped(lib):
    cfg = CONFIGS[0]
    x, w, ref = cfg_reference(cfg)
    d = lib.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad, cfg.dilation, cfg.shift,
                      out_mode=3)
    try:
        lib.test_fail_nth_encode(1)                  # the weight tensor map of the plan
        with pytest.raises(b2c.B2CError) as err:
            lib.Plan(d, b2c.POLICY_MIN_OVERHEAD)
        assert err.value.code == b2c.E_CUDA
        lib.test_fail_nth_encode(1)                  # first candidate of the timed selection cannot be built:
        plan = lib.Plan(d, b2c.POLICY_AUTO_TIMED)    # it is left out, the others are still timed
        lib.test_fail_nth_encode(0)
        cp = [e.id for e in lib.enumerate_embeddings(d) if e.variant == b2c.VARIANT_CP_TMA][0]
        plan2 = lib.Plan(d, cp)
        plan2.set_weights(to_dev(w))
        ws2 = torch.zeros(max(16, plan2.workspace_bytes()), dtype=torch.uint8, device="cuda")
        y32 = torch.zeros(ref[0].shape, dtype=torch.int32, device="cuda")
        y8 = torch.zeros(ref[1].shape, dtype=torch.int8, device="cuda")
        lib.test_fail_nth_encode(1)                  # the activation tensor map of a run
        with pytest.raises(b2c.B2CError) as err:
            plan2.run(to_dev(x), y32, y8, ws2)
        assert err.value.code == b2c.E_CUDA
        plan2.run(to_dev(x), y32, y8, ws2)           # the next run is not affected
        torch.cuda.synchronize()
        assert np.array_equal(y32.cpu().numpy(), ref[0])
        plan2.destroy()
    finally:
        lib.test_fail_nth_encode(0)
    assert plan.info().device_us > 0
    plan.set_weights(to_dev(w))
    y32 = torch.zeros(ref[0].shape, dtype=torch.int32, device="cuda")
    y8 = torch.zeros(ref[1].shape, dtype=torch.int8, device="cuda")
    ws = torch.zeros(max(16, plan.workspace_bytes()), dtype=torch.uint8, device="cuda")
    plan.run(to_dev(x), y32, y8, ws)
    torch.cuda.synchronize()
    assert np.array_equal(y32.cpu().numpy(), ref[0]) and np.array_equal(y8.cpu().numpy(), ref[1])
    plan.destroy()


# ---- issue-rate measurement of the intrinsic ------------------------------------------------------------
def test_mma_rate_measurement_is_plausible(lib):
    us, cyc = lib.measure_mma_rate(256, 4000)
    # a 128 x 256 x 32 int8 MMA cannot take fewer cycles than 8192 MACs per clock per SM would allow
    assert 100.0 < cyc < 400.0 and us > 0
    us16, cyc16 = lib.measure_mma_rate(16, 4000)
    assert cyc16 < cyc
    with pytest.raises(b2c.B2CError):
        lib.measure_mma_rate(48, 4000)
    # two-SM form: 256 x 256 x 32 per instruction; a pair cannot beat two SMs' worth of MACs per clock
    us2, cyc2 = lib.measure_mma_rate_pair(256, 4000)
    assert 100.0 < cyc2 < 600.0 and us2 > 0
    with pytest.raises(b2c.B2CError):
        lib.measure_mma_rate_pair(32, 4000)


# ---- failure detection: a wait that cannot complete ends by itself and is reported --------------------
def test_pack_kernel_wait_reports_timeout(lib):
    d = lib.make_desc(1, 32, 8, 8, 16, 3, 3, 1, 1, 1, 0, out_mode=1)
    plan = lib.Plan(d, b2c.POLICY_MIN_OVERHEAD)
    plan.selftest_pack_wait()               # waits for bytes that no copy delivers: gives up after its limit
    torch.cuda.synchronize()
    assert plan.device_status() == b2c.E_TIMEOUT
    assert plan.device_status() == b2c.OK
    plan.destroy()



def test_bounded_wait_reports_timeout_and_plan_stays_usable(lib):
    cfg = CONFIGS[0]
    x, w, ref = cfg_reference(cfg)
    d = lib.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad, cfg.dilation, cfg.shift,
                      out_mode=3)
    plan = lib.Plan(d, b2c.POLICY_MIN_OVERHEAD)
    plan.set_weights(to_dev(w))
    plan.selftest_bounded_wait()            # waits on a barrier nothing completes: gives up after its limit
    torch.cuda.synchronize()
    assert plan.device_status() == b2c.E_TIMEOUT
    assert plan.device_status() == b2c.OK   # the status word is cleared by the read
    y32 = torch.zeros(ref[0].shape, dtype=torch.int32, device="cuda")
    y8 = torch.zeros(ref[0].shape, dtype=torch.int8, device="cuda")
    ws = torch.zeros(max(16, plan.workspace_bytes()), dtype=torch.uint8, device="cuda")
    plan.run(to_dev(x), y32, y8, ws)        # the context and the plan still work
    torch.cuda.synchronize()
    assert plan.device_status() == b2c.OK
    assert np.array_equal(y32.cpu().numpy(), ref[0]) and np.array_equal(y8.cpu().numpy(), ref[1])
    plan.destroy()


# ---- degenerate and extreme shapes ----------------------------------------------------------------------
_EDGE = [
    # N, C, H, W, K, R, S, stride, pad, dil, shift
    (1, 1, 1, 1, 1, 1, 1, 1, 0, 1, 0),            # a single multiply
    (3, 2, 1, 1, 5, 3, 3, 1, 1, 1, 2),            # 1x1 image, every tap but the centre is padding
    (2, 4, 5, 7, 3, 5, 7, 1, 0, 1, 4),            # kernel as large as the image: P = Q = 1
    (40, 3, 3, 3, 9, 2, 2, 1, 0, 1, 3),           # P*Q = 4: one tile spans 32 images
    (1, 8, 9, 9, 4, 2, 2, (4, 5), 0, 1, 1),       # stride larger than the kernel
    (1, 2, 20, 20, 6, 3, 3, 1, 6, (7, 5), 5),     # dilation wider than half the image, pad 6
    (2, 32, 4, 4, 7, 1, 1, 1, 0, 1, 6),           # C*R*S exactly one MMA K step
    (1, 43, 5, 5, 33, 3, 1, 1, (1, 0), 1, 7),     # C*R*S = 129: one byte into the second 128-byte block
    (1, 131071, 1, 2, 2, 1, 1, 1, 0, 1, 20),      # the largest reduction length the library accepts
    (1, 1, 3, 300, 2, 1, 280, 1, 0, 1, 8),        # one very wide run of taps
]


@pytest.mark.parametrize("case", _EDGE, ids=lambda c: "n%dc%dh%dw%dk%dr%ds%d" % c[:7])
def test_edge_shapes(lib, case):
    N, C, H, W, K, R, S, stride, pad, dil, shift = case
    x = int8_uniform((N, C, H, W), 811)
    w = int8_uniform((K, C, R, S), 812)
    ref = oracle.conv2d_int8(x, w, stride, pad, dil, shift)
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, dil, shift, out_mode=3)
    embs = lib.enumerate_embeddings(d)
    assert embs
    done = set()
    for e in embs:
        key = (e.variant, e.split_k > 1)
        if key in done:
            continue
        done.add(key)
        check_against_oracle(x, w, stride, pad, dil, shift, 3, e.id, ref=ref)


def test_large_grid_staged_window_walks_tiles(lib):
    # 980 tiles of a low-channel strided shape: the staged-window kernel runs persistently
    N, C, H, W, K, R, S = 10, 3, 224, 224, 64, 7, 7
    x = int8_uniform((N, C, H, W), 711)
    w = int8_uniform((K, C, R, S), 712)
    ref = oracle.conv2d_int8(x, w, 2, 3, 1, 7)
    d = lib.make_desc(N, C, H, W, K, R, S, 2, 3, 1, 7, out_mode=3)
    for tile_n in (32, 64):
        ids = [e.id for e in lib.enumerate_embeddings(d) if e.variant == 3 and e.tile_n == tile_n and e.split_k == 1]
        assert ids
        check_against_oracle(x, w, 2, 3, 1, 7, 3, ids[0], ref=ref)


# ---- streaming host-buffer calls: copy in, path and copy out of successive calls overlap ----------
@pytest.mark.parametrize("policy", [b2c.POLICY_MIN_OVERHEAD, b2c.POLICY_AUTO_TIMED])
def test_streaming_host_calls(lib, policy):
    """Eleven calls with different inputs through a ring of three device buffer sets: every output must be
    the oracle's for ITS input (a slot reused too early, or a read-back that overtakes its kernel, breaks one)."""
    N, C, H, W, K, R, S, stride, pad, shift = 3, 24, 19, 17, 40, 3, 3, 2, 1, 6
    d = lib.make_desc(N, C, H, W, K, R, S, stride, pad, shift=shift, out_mode=3)
    w = int8_uniform((K, C, R, S), 911)
    plan = lib.Plan(d, policy)
    raw = lib.load()
    plan.host_sync()  # nothing enqueued yet: returns at once
    xs = [torch.from_numpy(int8_uniform((N, C, H, W), 920 + i)).pin_memory().numpy() for i in range(11)]
    P, Q = lib.out_shape(d)
    y32 = [torch.zeros((N, K, P, Q), dtype=torch.int32).pin_memory().numpy() for _ in xs]
    y8 = [torch.zeros((N, K, P, Q), dtype=torch.int8).pin_memory().numpy() for _ in xs]
    hp = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    assert raw.b2c_plan_run_host_async(plan._h, hp(xs[0]), hp(y32[0]), hp(y8[0])) == b2c.E_NOT_READY
    plan.set_weights(to_dev(w))
    torch.cuda.synchronize()
    assert raw.b2c_plan_run_host_async(plan._h, hp(xs[0]), None, hp(y8[0])) == b2c.E_INVALID_ARG
    assert raw.b2c_plan_run_host_async(plan._h, None, hp(y32[0]), hp(y8[0])) == b2c.E_INVALID_ARG
    for i, x in enumerate(xs):
        plan.run_host_async(x, y32[i], y8[i])
    plan.host_sync()
    for i, x in enumerate(xs):
        want32, want8 = oracle.conv2d_int8(x, w, stride, pad, 1, shift)
        assert np.array_equal(y32[i], want32), i
        assert np.array_equal(y8[i], want8), i
    assert plan.device_status() == b2c.OK
    # pageable host memory: same results (the copies are then synchronous)
    xp = int8_uniform((N, C, H, W), 990)
    o32 = np.zeros((N, K, P, Q), dtype=np.int32)
    o8 = np.zeros((N, K, P, Q), dtype=np.int8)
    plan.run_host_async(xp, o32, o8)
    plan.host_sync()
    want32, want8 = oracle.conv2d_int8(xp, w, stride, pad, 1, shift)
    assert np.array_equal(o32, want32) and np.array_equal(o8, want8)
    plan.destroy()


def test_streaming_host_calls_grouped(lib):
    N, C, H, W, K, R, S, groups = 2, 32, 12, 12, 32, 3, 3, 4
    d = lib.make_desc(N, C, H, W, K, R, S, 1, 1, out_mode=1)
    w = int8_uniform((K, C // groups, R, S), 931)
    plan = lib.Plan(d, groups=groups)
    plan.set_weights(to_dev(w))
    torch.cuda.synchronize()
    xs = [torch.from_numpy(int8_uniform((N, C, H, W), 940 + i)).pin_memory().numpy() for i in range(5)]
    ys = [torch.zeros((N, K, H, W), dtype=torch.int32).pin_memory().numpy() for _ in xs]
    for x, y in zip(xs, ys):
        plan.run_host_async(x, y)
    plan.host_sync()
    for x, y in zip(xs, ys):
        assert np.array_equal(y, oracle.conv2d_int8(x, w, 1, 1, 1, 0, groups=groups)[0])
    plan.destroy()
