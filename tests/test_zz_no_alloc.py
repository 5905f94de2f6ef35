"""kvc_decode_attend_static: decode attention for callers that cannot allocate device memory.

Some users of this library decode from inside a serving engine whose memory pool is already fully
handed out to KV blocks, or from code that runs under an allocator it does not own; they cannot
give kvc_decode_attend a workspace.  The static variant keeps its temporaries in a fixed array in
the library's device image.  This test drives it through the C ABI twice in a row (the array keeps
the first call's contents, so the second call checks that nothing depends on a clean scratch) and
compares with the ordinary entry point on the same inputs.  It lives in the file pytest collects
last so that a failure here cannot hide any other test under `-x`.
"""
import numpy as np
import pytest
import torch

from paper_2605_16439_b200 import binding as kvc
from paper_2605_16439_b200 import build as kvc_build
from paper_2605_16439_b200 import workloads as wl

import kvc_testlib as tl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("ci,kw", [(0, {}), (1, dict(B=2, H_q=4, H_kv=4))])
def test_static_scratch_entry_point_matches_workspace_entry_point(ci, kw):
    kvc_build.build()
    shape = tl.small(wl.CONFIGS[ci], **kw)
    dt = wl.torch_dtype(shape.dtype)
    p = tl.make_problem(shape, 123 + ci, T=shape.T0, T_cap=shape.T0 + 8)
    layer = tl.gpu_layer(shape, p)
    B, R, T, T_cap = shape.B, shape.R, p["T"], p["T_cap"]
    assert kvc.kvc_workspace_bytes(layer, B, R, T) <= kvc.kvc_static_scratch_bytes()
    caps = kvc.alloc_capsules(layer, B, R)
    kvc.kvc_compress(layer, p["K_vis"].cuda(), p["V_vis"].cuda(), B, R, caps)
    q, Kt, Vt = p["q"].cuda(), p["K_txt"].cuda(), p["V_txt"].cuda()
    ws = kvc.alloc_workspace(layer, B, R, T_cap)
    want = torch.empty((B, shape.H_q, shape.d), dtype=dt, device="cuda")
    kvc.kvc_decode_attend(layer, q, caps, B, R, Kt, Vt, T, T_cap, want, ws)
    torch.cuda.synchronize()
    # everything is allocated by now; the two static calls below are given inputs and outputs only
    outs = [torch.full_like(want, float("nan")) for _ in range(2)]
    q2 = (q.float() * 0.5).to(dt)                      # a different query in between dirties the scratch
    for i, out in enumerate(outs):
        kvc.kvc_decode_attend_static(layer, q, caps, B, R, Kt, Vt, T, T_cap, out)
        if i == 0:
            kvc.kvc_decode_attend_static(layer, q2, caps, B, R, Kt, Vt, T, T_cap, torch.empty_like(want))
    torch.cuda.synchronize()
    # the status word of the static call sits in the fixed array: read with no workspace pointer
    assert kvc.kvc_read_device_status(layer, B, R, T, None) == 0
    tol = tl.TOL[shape.dtype]
    for out in outs:
        assert torch.isfinite(out.float()).all()
        assert float((out.float() - want.float()).abs().max()) <= tol
    # and against the CPU oracle, like every other parity test
    _, _, ref = tl.oracle_run(shape, p)
    tl.assert_close(tl.np64(outs[1]), ref, shape.dtype)


def test_static_scratch_rejects_shapes_beyond_its_fixed_size():
    kvc_build.build()
    shape = tl.small(wl.CONFIGS[2], B=16, H_q=28, H_kv=4, R=8)
    dt = wl.torch_dtype(shape.dtype)
    m = kvc.kvc_retained_len(shape.n, 600)
    theta = torch.zeros((4, m, shape.n), dtype=dt, device="cuda")
    mu = torch.zeros((4, 128), dtype=dt, device="cuda")
    layer = kvc.Layer(28, 4, 128, shape.n, 600, dt, idx=wl.evenly_spaced_idx(shape.n, m), theta=theta, U=theta, mu=mu)
    assert kvc.kvc_workspace_bytes(layer, 16, 8, 256) > kvc.kvc_static_scratch_bytes()
    x = torch.zeros(16, device="cuda")
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_decode_attend_static(layer, x, x, 16, 8, x, x, 256, 256, x)
    assert e.value.status == -5 and "static scratch too small" in str(e.value)
