"""Helpers for the GPU parity tests: run one embedding through the C ABI and fetch the outputs."""
import numpy as np
import torch

import oracle
import paper_2104_04731_b200 as b2c


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run_embedding(x, w, stride, pad, dilation, shift, out_mode, policy_or_id, in_layout=b2c.LAYOUT_NCHW,
                  out_layout=b2c.LAYOUT_NCHW):
    """x NCHW int8 numpy, w KCRS int8 numpy.  Returns (y32, y8, embedding) with outputs as NKPQ numpy."""
    N, C, H, W = x.shape
    K, _, R, S = w.shape
    d = b2c.make_desc(N, C, H, W, K, R, S, stride, pad, dilation, shift, in_layout, out_layout, out_mode)
    P, Q = b2c.out_shape(d)
    plan = b2c.Plan(d, policy_or_id)
    try:
        emb = plan.info()
        xin = x if in_layout == b2c.LAYOUT_NCHW else x.transpose(0, 2, 3, 1)
        xd, wd = to_dev(xin), to_dev(w)
        oshape = (N, K, P, Q) if out_layout == b2c.LAYOUT_NCHW else (N, P, Q, K)
        # poison the outputs so that unwritten elements show up
        y32 = torch.full(oshape, -7777777, dtype=torch.int32, device="cuda") if out_mode & 1 else None
        y8 = torch.full(oshape, 77, dtype=torch.int8, device="cuda") if out_mode & 2 else None
        ws_bytes = plan.workspace_bytes()
        ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
        ws.fill_(0xAB)
        plan.set_weights(wd)
        plan.run(xd, y32, y8, ws)
        torch.cuda.synchronize()
        assert plan.device_status() == b2c.OK

        def back(t):
            if t is None:
                return None
            a = t.cpu().numpy()
            return a if out_layout == b2c.LAYOUT_NCHW else np.ascontiguousarray(a.transpose(0, 3, 1, 2))

        return back(y32), back(y8), emb
    finally:
        plan.destroy()


def check_against_oracle(x, w, stride, pad, dilation, shift, out_mode, policy_or_id, ref=None, **kw):
    if ref is None:
        ref = oracle.conv2d_int8(x, w, stride, pad, dilation, shift)
    y32, y8, emb = run_embedding(x, w, stride, pad, dilation, shift, out_mode, policy_or_id, **kw)
    tag = "variant=%d tile_n=%d split_k=%d" % (emb.variant, emb.tile_n, emb.split_k)
    if out_mode & 1:
        bad = int((y32 != ref[0]).sum())
        assert bad == 0, "%s: %d of %d int32 outputs differ" % (tag, bad, ref[0].size)
    if out_mode & 2:
        bad = int((y8 != ref[1]).sum())
        assert bad == 0, "%s: %d of %d int8 outputs differ" % (tag, bad, ref[1].size)
    return emb
