"""The bounds-checked build of the library (libb2conv_debug.so, the same sources with -DB2C_DEBUG_BOUNDS).

It stands in for a memory checker: every address a kernel computes by hand is tested against its
tensor's range, and the workspace sits between two guard bands.  The GPU test runs the five benchmark
shapes through every layout variant in that build (a child process, because the binding picks its
library when it is first loaded): no report, guard bands intact, outputs equal to the oracle's.  It
then declares every range 64 bytes too short: the accesses to the last elements, which are in range,
must be reported with their site and skipped, and nothing else may change.
"""
import ctypes
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import sys
import numpy as np
import torch
import oracle
import paper_2104_04731_b200 as b2c
from paper_2104_04731_b200.synth import CONFIGS, int8_uniform

assert b2c.debug_build()
runs = 0
for cfg in CONFIGS:
    x, w = cfg.tensors()
    ref32, ref8 = oracle.conv2d_int8(x, w, cfg.stride, cfg.pad, cfg.dilation, cfg.shift)
    d = b2c.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad, cfg.dilation, cfg.shift, out_mode=3)
    xd, wd = torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda()
    seen = set()
    for e in b2c.enumerate_embeddings(d):
        key = (e.variant, e.tile_m, e.map_m, min(e.split_k, 2))
        if key in seen:
            continue
        seen.add(key)
        plan = b2c.Plan(d, e.id)
        y32 = torch.full(ref32.shape, -7777777, dtype=torch.int32, device="cuda")
        y8 = torch.full(ref8.shape, 77, dtype=torch.int8, device="cuda")
        ws = torch.zeros(max(16, plan.workspace_bytes()), dtype=torch.uint8, device="cuda")
        plan.set_weights(wd)
        plan.run(xd, y32, y8, ws)
        st = plan.device_status()
        assert st == b2c.OK, (cfg.name, e.variant, e.tile_n, st, plan.debug_info())
        assert plan.canaries_intact(ws), (cfg.name, e.variant)
        assert np.array_equal(y32.cpu().numpy(), ref32) and np.array_equal(y8.cpu().numpy(), ref8), (cfg.name, e.variant)
        plan.destroy()
        runs += 1

# every range declared 64 bytes short: the last elements are reported and skipped, the rest is written
cfg = CONFIGS[0]
x, w = cfg.tensors()
ref32, ref8 = oracle.conv2d_int8(x, w, cfg.stride, cfg.pad, cfg.dilation, cfg.shift)
d = b2c.make_desc(cfg.N, cfg.C, cfg.H, cfg.W, cfg.K, cfg.R, cfg.S, cfg.stride, cfg.pad, cfg.dilation, cfg.shift, out_mode=3)
sites = set()
for e in b2c.enumerate_embeddings(d):
    if e.split_k != 1 or e.variant in sites:
        continue
    plan = b2c.Plan(d, e.id)
    plan.set_weights(torch.from_numpy(w).cuda())
    y32 = torch.full(ref32.shape, -7777777, dtype=torch.int32, device="cuda")
    y8 = torch.full(ref8.shape, 77, dtype=torch.int8, device="cuda")
    ws = torch.zeros(max(16, plan.workspace_bytes()), dtype=torch.uint8, device="cuda")
    b2c.test_shrink_checked_ranges(64)
    plan.run(torch.from_numpy(x).cuda(), y32, y8, ws)
    st = plan.device_status()
    b2c.test_shrink_checked_ranges(0)
    site, off = plan.debug_info()
    assert st == b2c.E_BOUNDS and site > 0, (e.variant, st, site, off)
    got = y8.cpu().numpy().ravel()
    # the last 64 int8 outputs may be missing, nothing before them may differ from the oracle unless a
    # skipped load or scratch store fed it (layout variants): those only ever zero or drop data, so the
    # untouched poison value 77 or a wrong value can appear, but never a write outside the tensor
    assert plan.canaries_intact(ws)
    plan.run(torch.from_numpy(x).cuda(), y32, y8, ws)   # ranges restored: clean again
    assert plan.device_status() == b2c.OK
    assert np.array_equal(y32.cpu().numpy(), ref32) and np.array_equal(y8.cpu().numpy(), ref8)
    plan.destroy()
    sites.add(e.variant)
print("debug build ok: %d runs, shrink reported for variants %s" % (runs, sorted(sites)))
'''


def test_debug_library_exports_the_same_interface():
    from paper_2104_04731_b200 import build
    import paper_2104_04731_b200 as b2c

    lib = ctypes.CDLL(build.build(debug=True))
    for name in b2c.EXPORTS:
        assert hasattr(lib, name), name
    assert lib.b2c_debug_build() == 1
    assert b2c.load().b2c_debug_build() == (1 if os.environ.get("B2C_DEBUG_LIB") == "1" else 0)


@pytest.mark.gpu
def test_five_shapes_through_the_bounds_checked_build():
    env = dict(os.environ, B2C_DEBUG_LIB="1", PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "debug build ok" in r.stdout
