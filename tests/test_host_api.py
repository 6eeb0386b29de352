"""Host-side logic of the GPU library that needs no device: exported symbols, descriptor
validation, output shapes and the embedding planner's enumeration and overhead terms."""
import ctypes
import os
import re

import pytest

import oracle
import paper_2104_04731_b200 as b2c
from paper_2104_04731_b200.synth import CONFIGS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2104_04731_b200 import build

    build.build()
    return b2c.load()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "b2conv.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(b2c_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations parsed"
    assert declared == set(b2c.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert b2c.status_string(0) == "ok"
    for code in range(-6, 0):
        assert b2c.status_string(code) not in ("ok", "unknown status")
    assert b2c.status_string(-99) == "unknown status"


@pytest.mark.parametrize("cfg", CONFIGS, ids=lambda c: c.name)
def test_out_shape_matches_oracle_formula(lib, cfg):
    d = b2c.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad, cfg.dilation)
    assert b2c.out_shape(d) == oracle.out_shape(cfg.H, cfg.W, cfg.R, cfg.S, cfg.stride, cfg.pad, cfg.dilation)
    assert b2c.out_shape(d) == (cfg.P, cfg.Q)


def test_out_shape_odd_cases(lib):
    for (H, W, R, S, st, pd, dl) in [(5, 7, 3, 3, (2, 3), (0, 1), (2, 1)), (9, 9, 2, 4, (3, 1), (2, 0), (1, 2)), (4, 4, 3, 3, 1, 0, 2)]:
        d = b2c.make_desc(1, 1, H, W, 1, R, S, st, pd, dl)
        assert b2c.out_shape(d) == oracle.out_shape(H, W, R, S, st, pd, dl)


def test_descriptor_validation(lib):
    good = dict(N=1, C=4, H=8, W=8, K=4, R=3, S=3)
    n = ctypes.c_int32()
    for bad in [dict(N=0), dict(C=0), dict(K=-1), dict(R=0), dict(stride=0), dict(pad=-1), dict(dilation=0),
                dict(shift=32), dict(shift=-1), dict(in_layout=2), dict(out_layout=5), dict(out_mode=0), dict(out_mode=4)]:
        d = b2c.make_desc(**{**good, **bad})
        assert lib.b2c_enumerate(ctypes.byref(d), None, 0, ctypes.byref(n)) == b2c.E_INVALID_ARG, bad
    # kernel larger than the padded image: empty output
    d = b2c.make_desc(1, 1, 2, 2, 1, 5, 5)
    assert lib.b2c_enumerate(ctypes.byref(d), None, 0, ctypes.byref(n)) == b2c.E_UNSUPPORTED
    # C*R*S above 131071 could overflow an int32 accumulator
    d = b2c.make_desc(1, 131072, 1, 1, 1, 1, 1)
    assert lib.b2c_enumerate(ctypes.byref(d), None, 0, ctypes.byref(n)) == b2c.E_UNSUPPORTED
    d = b2c.make_desc(1, 131071, 1, 1, 1, 1, 1)
    assert lib.b2c_enumerate(ctypes.byref(d), None, 0, ctypes.byref(n)) == b2c.OK
    # null pointers
    assert lib.b2c_enumerate(None, None, 0, ctypes.byref(n)) == b2c.E_INVALID_ARG
    assert lib.b2c_out_shape(None, None, None) == b2c.E_INVALID_ARG
    assert lib.b2c_plan_info(None, None) == b2c.E_INVALID_ARG
    assert lib.b2c_conv2d_int8_run(None, None, None, None, None, None) == b2c.E_INVALID_ARG
    assert lib.b2c_conv2d_int8(1, 1, 4, 4, 1, 1, 1, 1, 0, 1, 0, None, None, None, None, None) == b2c.E_INVALID_ARG


@pytest.mark.parametrize("cfg", CONFIGS, ids=lambda c: c.name)
def test_enumeration_is_sorted_and_covers_variants(lib, cfg):
    d = b2c.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad, cfg.dilation, cfg.shift,
                      out_mode=cfg.out_mode)
    embs = b2c.enumerate_embeddings(d)
    assert embs
    assert [e.id for e in embs] == list(range(len(embs)))
    costs = [e.o_mac + e.o_data for e in embs]
    assert costs == sorted(costs)
    assert {0, 1, 2} <= {e.variant for e in embs} <= {0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10}
    for e in embs:
        assert e.tile_m in (128, 256) and e.tile_n in (16, 32, 64, 128, 256) and e.split_k >= 1
        if e.tile_m == 256:   # two-SM schedule: TMA-fed maps, no split, column tile of at least 32
            assert e.variant in (0, 1, 4, 5, 6) and e.split_k == 1 and e.tile_n >= 32 and e.map_m == b2c.AXIS_NPQ
        assert (e.map_m, e.map_n) in ((b2c.AXIS_NPQ, b2c.AXIS_K), (b2c.AXIS_K, b2c.AXIS_NPQ))
        if e.map_m == b2c.AXIS_K:  # swapped map: TMA-fed variants only, and only when K fills half a tile
            assert e.variant in (0, 1, 4, 5) and cfg.K >= 64 and e.tile_n >= 32
        assert e.map_k == {0: b2c.AXIS_C, 6: b2c.AXIS_C, 7: b2c.AXIS_C, 4: b2c.AXIS_SC, 9: b2c.AXIS_SC, 5: b2c.AXIS_C_PHASES, 8: b2c.AXIS_C_PHASES}.get(e.variant, b2c.AXIS_CRS)
        assert e.o_mac >= 0 and e.o_data >= 0 and e.device_us == -1.0
        if e.variant in (b2c.VARIANT_IM2COL_GATHER, b2c.VARIANT_IM2COL_STAGED, b2c.VARIANT_IM2COL_WINDOW) and e.split_k == 1:
            assert e.workspace_bytes == 0


def test_channel_pack_utilisation_law(lib):
    # Section 6.1: with ic < z only ic/z of the intrinsic's work is useful.  With M a multiple
    # of 128 and K equal to the tile width, MAC_total / MAC_min must equal C_pad / C exactly.
    for C, C_pad in [(1, 32), (3, 32), (16, 32), (32, 32), (33, 64), (72, 96)]:
        N, H, W, K, R, S = 2, 16, 16, 64, 3, 3  # pad 1 stride 1 -> P = Q = 16, M = 512
        d = b2c.make_desc(N, C, H, W, K, R, S, 1, 1, 1)
        mac_min = N * K * 16 * 16 * C * R * S
        cp = [e for e in b2c.enumerate_embeddings(d)
              if e.variant == 0 and e.tile_n == 64 and e.split_k == 1 and e.map_m == b2c.AXIS_NPQ]
        assert sorted(e.tile_m for e in cp) == [128, 256]   # one-SM and two-SM schedule of the same map
        for e in cp:                                        # M = 512 is a multiple of both tile heights
            assert (e.o_mac + mac_min) * C == mac_min * C_pad
        # the stencil-unroll maps pad the fused (c, r, s) axis to 32 instead
        kp = -(-C * R * S // 32) * 32
        un = [e for e in b2c.enumerate_embeddings(d) if e.variant == 2 and e.tile_n == 64 and e.split_k == 1]
        assert (un[0].o_mac + mac_min) * (C * R * S) == mac_min * kp
        # swapped map (M <- k, N <- pixels): K = 64 fills half of the 128 accumulator rows, so the
        # issued MACs double on top of the channel padding; M = 512 pixels is a multiple of every tile
        for e in b2c.enumerate_embeddings(d):
            if e.variant == 0 and e.map_m == b2c.AXIS_K and e.split_k == 1:
                assert (e.o_mac + mac_min) * C == 2 * mac_min * C_pad


def test_padding_inflates_weights_and_workspace(lib):
    # Section 6.1: padding ic inflates the weight tensor as well; here it shows in o_data and in
    # the scratch size of the channel-pack map.
    cfg = CONFIGS[2]  # C = 3
    d = b2c.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad)
    embs = [e for e in b2c.enumerate_embeddings(d) if e.map_m == b2c.AXIS_NPQ]
    cp = next(e for e in embs if e.variant == 0 and e.split_k == 1)
    ga = next(e for e in embs if e.variant == 2 and e.split_k == 1)
    ex = next(e for e in embs if e.variant == 1 and e.split_k == 1)
    assert cp.workspace_bytes == cfg.N * cfg.H * cfg.W * 32
    assert ex.workspace_bytes == cfg.N * cfg.P * cfg.Q * 160
    assert ga.workspace_bytes == 0
    assert ga.o_mac < cp.o_mac and ga.o_data < ex.o_data < cp.o_data + ex.o_data
    # partial unroll (Table 2: stencil unroll on one axis only) and image pack sit between the two
    ro = next(e for e in embs if e.variant == 4 and e.split_k == 1)
    sd = next(e for e in embs if e.variant == 5 and e.split_k == 1)
    assert ro.workspace_bytes == cfg.N * cfg.H * cfg.Q * 32          # (s, c) = 21 -> 32 channels per (n, h, q)
    # 3*2*2 = 12 phase bytes per column: two columns share a 32-byte pixel, so R' = 4 and S' = 4 -> 2 taps at
    # dilation 2 over Q + 2 scratch columns; scratch sizes are rounded up to 256 bytes
    assert sd.workspace_bytes == -(-cfg.N * (cfg.P + 3) * (cfg.Q + 2) * 32 // 256) * 256
    # single channel, 9 x 21 stride 2: 4 phase bytes per column, so eight columns share a 32-byte pixel and the
    # S' = 11 taps of a row become 2 taps at dilation 8 over Q + 8 scratch columns (R' = 5)
    c4 = CONFIGS[3]
    d4 = b2c.make_desc(c4.N, c4.C, c4.H, c4.W, c4.K, c4.R, c4.S, c4.stride, c4.pad)
    sd4 = next(e for e in b2c.enumerate_embeddings(d4) if e.variant == 5 and e.split_k == 1)
    assert sd4.workspace_bytes == -(-c4.N * (c4.P + 4) * (c4.Q + 8) * 32 // 256) * 256
    assert ga.o_mac < ro.o_mac < cp.o_mac
    assert embs[0].variant in (2, 3)  # lowest overhead: stencil unroll formed inside the kernel


def test_nhwc_input_channel_pack_scratch(lib):
    # 24 channels: the NHWC input is re-padded to 32 in the scratch tensor; 64 channels: read in place
    d = b2c.make_desc(1, 24, 8, 8, 16, 3, 3, 1, 1, in_layout=b2c.LAYOUT_NHWC)
    cp = [e for e in b2c.enumerate_embeddings(d) if e.variant == 0 and e.split_k == 1 and e.tile_m == 128]
    assert cp and all(e.workspace_bytes == 256 * -(-(8 * 8 * 32) // 256) for e in cp)
    d = b2c.make_desc(1, 64, 8, 8, 16, 3, 3, 1, 1, in_layout=b2c.LAYOUT_NHWC)
    cp = [e for e in b2c.enumerate_embeddings(d) if e.variant == 0 and e.split_k == 1]
    assert cp and all(e.workspace_bytes == 0 for e in cp)


def test_swapped_map_is_listed_only_when_k_fills_half_a_tile(lib):
    for K, listed in [(16, False), (63, False), (64, True), (129, True), (512, True)]:
        d = b2c.make_desc(2, 32, 12, 12, K, 3, 3, 1, 1)
        swapped = [e for e in b2c.enumerate_embeddings(d) if e.map_m == b2c.AXIS_K]
        assert bool(swapped) == listed, K
        for e in swapped:
            assert e.map_n == b2c.AXIS_NPQ and e.variant in (0, 1, 4, 5)
            # pixel tile: covering width or less than a quarter of its columns wasted
            M = 2 * 12 * 12
            n_pad = -(-M // e.tile_n) * e.tile_n
            assert e.tile_n >= M or e.tile_n == 256 or (n_pad - M) * 4 <= n_pad
            # a swapped split reduction meets in memory: int8 output needs the int32 scratch
            if e.split_k > 1:
                d8 = b2c.make_desc(2, 32, 12, 12, K, 3, 3, 1, 1, out_mode=2)
                e8 = next(c for c in b2c.enumerate_embeddings(d8)
                          if (c.map_m, c.variant, c.tile_n, c.split_k) == (e.map_m, e.variant, e.tile_n, e.split_k))
                assert e8.workspace_bytes >= 4 * M * K


def test_output_extent_overflow_is_refused(lib):
    # small image, huge padding: P = Q = 61000, P*Q beyond 31 bits
    d = b2c.make_desc(1, 1, 1000, 1000, 1, 1, 1, 1, 30000, 1)
    n = ctypes.c_int32()
    assert b2c.load().b2c_enumerate(ctypes.byref(d), None, 0, ctypes.byref(n)) == b2c.E_UNSUPPORTED
    # padding beyond any use
    d = b2c.make_desc(1, 1, 8, 8, 1, 3, 3, 1, (1 << 20) + 1, 1)
    assert b2c.load().b2c_enumerate(ctypes.byref(d), None, 0, ctypes.byref(n)) == b2c.E_UNSUPPORTED
    # a large but representable extent is still listed
    d = b2c.make_desc(1, 1, 1000, 1000, 1, 1, 1, 1, 5000, 1)
    assert b2c.load().b2c_enumerate(ctypes.byref(d), None, 0, ctypes.byref(n)) == b2c.OK and n.value > 0


def test_fault_injection_hook_arms_and_disarms(lib):
    assert b2c.load().b2c_test_fail_nth_encode(-1) == b2c.E_INVALID_ARG
    b2c.test_fail_nth_encode(3)
    b2c.test_fail_nth_encode(0)
