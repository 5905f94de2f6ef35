"""Batches with per-sequence lengths: the CUDA path against the oracle's masked formulation, through the C ABI.

The lengths live in device arrays the kernels read.  Storage a sequence does not have (blocks >= R_b[b], text rows
>= T_b[b]) is filled with NaN before the decode call, so any read of it that reaches a result shows.
"""
import numpy as np
import pytest
import torch

from oracle import kvcapsule_oracle as orc
from paper_2605_16439_b200 import binding as kvc
from paper_2605_16439_b200 import build as kvc_build
from paper_2605_16439_b200 import workloads as wl

import kvc_testlib as tl

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module", autouse=True)
def _built():
    kvc_build.build()


def _i32(x):
    return torch.tensor(list(x), dtype=torch.int32, device=DEV)


def _status(layer, B, R, T, ws):
    return kvc.kvc_read_device_status(layer, B, R, T, ws)


@pytest.mark.parametrize("grid", [12, 8, 16])          # n = 144: three-phase kernels; n = 64, 256 in bf16: the resident-parameter kernel
@pytest.mark.parametrize("mode", ["kv", "k", "v"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_mixed_block_counts_and_text_lengths_in_one_call(dtype, mode, grid):
    R_b = [0, 1, 5, 5, 1, 0, 0, 3]
    T_b = [1, 0, 257, 0, 257, 257, 0, 64]
    B, R_max, T_cap = len(R_b), 5, 300
    shape = wl.Shape("ragged", 1, B, 6, 2, 128, grid, R_max, T_cap, 1, dtype, 600)      # G = 3
    p = tl.make_problem(shape, 811, T=T_cap, T_cap=T_cap, recipe="peaked")
    layer = tl.gpu_layer(shape, p, DEV, mode)
    caps = kvc.alloc_capsules(layer, B, R_max, DEV)
    kvc.kvc_compress(layer, p["K_vis"].to(DEV), p["V_vis"].to(DEV), B, R_max, caps)
    K_g, V_g = kvc.capsule_views(layer, caps, B, R_max)
    K_txt, V_txt = p["K_txt"].to(DEV), p["V_txt"].to(DEV)
    for b in range(B):
        K_g[b, :, R_b[b]:] = float("nan")
        V_g[b, :, R_b[b]:] = float("nan")
        K_txt[b, :, T_b[b]:] = float("nan")
        V_txt[b, :, T_b[b]:] = float("nan")
    ws = kvc.alloc_workspace(layer, B, R_max, T_cap, DEV)
    ws.fill_(0xFF)                                       # NaN patterns: stale scratch must not matter either
    out = torch.full((B, shape.H_q, 128), float("nan"), dtype=wl.torch_dtype(dtype), device=DEV)
    kvc.kvc_profile_start(16)
    kvc.kvc_decode_attend_ragged(layer, p["q"].to(DEV), caps, B, R_max, _i32(R_b), K_txt, V_txt, max(T_b), _i32(T_b),
                                 T_cap, out, ws)
    torch.cuda.synchronize()
    kvc.kvc_profile_stop()
    launches = {k: v[1] for k, v in kvc.kvc_profile_read().items()}
    kvc.kvc_profile_start(0)
    kvc.kvc_profile_stop()
    # short blocks in bf16 take the resident-parameter kernel, which reads the lengths itself; everything else the three-phase kernels
    assert launches["resident"] == (1 if (dtype == "bf16" and mode == "kv" and grid in (8, 16)) else 0)
    assert launches["scores"] == 1 - launches["resident"]
    assert _status(layer, B, R_max, max(T_b), ws) == 0
    K_o, V_o = orc.compress(tl.np64(p["K_vis"]), tl.np64(p["V_vis"]), p["idx"].numpy(), tl.np64(p["U"]), tl.np64(p["mu"]),
                            shape.n, False, mode)
    want = orc.decode_attend_ragged(tl.np64(p["q"]), K_o, V_o, tl.np64(p["theta"]), tl.np64(p["U"]), tl.np64(p["mu"]),
                                    tl.np64(p["K_txt"]), tl.np64(p["V_txt"]), R_b, T_b, mode)
    got = tl.np64(out)
    assert not got[6].any()                              # the sequence without any row
    tl.assert_close(got, want, dtype, "ragged decode")
    # every sequence equals the uniform call made for it alone (same kernels or not: within the bound of both)
    for b in (2, 4):
        o1 = torch.empty((1, shape.H_q, 128), dtype=out.dtype, device=DEV)
        caps1 = kvc.alloc_capsules(layer, 1, R_b[b], DEV)
        kvc.kvc_compress(layer, p["K_vis"][b:b + 1, :, :R_b[b] * shape.n].contiguous().to(DEV),
                         p["V_vis"][b:b + 1, :, :R_b[b] * shape.n].contiguous().to(DEV), 1, R_b[b], caps1)
        ws1 = kvc.alloc_workspace(layer, 1, R_b[b], T_cap, DEV)
        kvc.kvc_decode_attend(layer, p["q"][b:b + 1].to(DEV), caps1, 1, R_b[b], p["K_txt"][b:b + 1].to(DEV),
                              p["V_txt"][b:b + 1].to(DEV), T_b[b], T_cap, o1, ws1)
        torch.cuda.synchronize()
        tl.assert_close(tl.np64(o1), want[b:b + 1], dtype, "the sequence alone")
    # NULL arrays mean the bounds for every sequence: the uniform call
    out_u = torch.empty_like(out)
    kvc.kvc_decode_attend_ragged(layer, p["q"].to(DEV), caps_full(layer, p, B, R_max), B, R_max, None, p["K_txt"].to(DEV),
                                 p["V_txt"].to(DEV), T_cap, None, T_cap, out_u, ws)
    torch.cuda.synchronize()
    want_u = orc.decode_attend_definition(tl.np64(p["q"]), K_o, V_o, tl.np64(p["theta"]), tl.np64(p["U"]), tl.np64(p["mu"]),
                                          tl.np64(p["K_txt"]), tl.np64(p["V_txt"]), False, mode)
    tl.assert_close(tl.np64(out_u), want_u, dtype, "uniform lengths")


def caps_full(layer, p, B, R):
    caps = kvc.alloc_capsules(layer, B, R, DEV)
    kvc.kvc_compress(layer, p["K_vis"].to(DEV), p["V_vis"].to(DEV), B, R, caps)
    return caps


@pytest.mark.parametrize("grid", [12, 16])
@pytest.mark.parametrize("mode", ["kv", "k", "v"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_ragged_compress_with_left_over_rows_then_decode(dtype, mode, grid):
    """Vision runs of 0, 1, 5 whole blocks and runs that are not a whole number of blocks: the left-over rows land in
    front of the text rows, bit-exact; the capsules of the whole blocks match the oracle; the decode on top matches."""
    n, R_max, T_cap = grid * grid, 5, grid * grid + 300
    N_v = [0, n, 5 * n, 2 * n + 7, 3, 2 * n + (n - 1), 4 * n + 64]
    T_own = [9, 0, 130, 1, 0, 257, 0]
    B = len(N_v)
    N_cap = 6 * n
    shape = wl.Shape("ragged", 1, B, 8, 2, 128, grid, 6, T_cap, 1, dtype, 600)
    p = tl.make_problem(shape, 907, T=T_cap, T_cap=T_cap, recipe="structured")
    dt = wl.torch_dtype(dtype)
    layer = tl.gpu_layer(shape, p, DEV, mode)
    K_vis, V_vis = p["K_vis"].to(DEV).clone(), p["V_vis"].to(DEV).clone()
    for b in range(B):
        K_vis[b, :, N_v[b]:] = float("nan")
        V_vis[b, :, N_v[b]:] = float("nan")
    caps = kvc.alloc_capsules(layer, B, R_max, DEV)
    caps.view(torch.int16).fill_(0x7FC0)                  # NaN in both storage types
    K_txt = torch.full((B, 2, T_cap, 128), float("nan"), dtype=dt, device=DEV)
    V_txt = torch.full_like(K_txt, float("nan"))
    R_b, T_b = torch.full((B,), -7, dtype=torch.int32, device=DEV), torch.full((B,), -7, dtype=torch.int32, device=DEV)
    kvc.kvc_compress_ragged(layer, K_vis, V_vis, B, N_cap, _i32(N_v), R_max, caps, K_txt, V_txt, T_cap, R_b, T_b)
    torch.cuda.synchronize()
    assert kvc.kvc_read_compress_status(layer) == 0
    K_o, V_o, R_o, K_tail, V_tail = orc.compress_ragged(tl.np64(p["K_vis"]), tl.np64(p["V_vis"]), N_v, p["idx"].numpy(),
                                                        tl.np64(p["U"]), tl.np64(p["mu"]), n, R_max, mode)
    assert R_b.tolist() == list(R_o) == [v // n for v in N_v]
    assert T_b.tolist() == [v % n for v in N_v]
    K_g, V_g = kvc.capsule_views(layer, caps, B, R_max)
    v_tol = (2e-5 if dtype == "f32" else 2.0 ** -8 + 2.0 ** -12) * max(1.0, float(np.abs(V_o).max()))
    for b in range(B):
        r, t = int(R_o[b]), N_v[b] % n
        assert np.array_equal(tl.np64(K_g[b, :, :r]), K_o[b, :, :r])
        assert np.abs(tl.np64(V_g[b, :, :r]) - V_o[b, :, :r]).max(initial=0.0) <= (0.0 if mode == "k" else v_tol)
        assert torch.isnan(K_g[b, :, r:].float()).all() and torch.isnan(V_g[b, :, r:].float()).all()   # left untouched
        assert np.array_equal(tl.np64(K_txt[b, :, :t]), K_tail[b]) and np.array_equal(tl.np64(V_txt[b, :, :t]), V_tail[b])
        assert torch.isnan(K_txt[b, :, t:].float()).all()
    # the caller appends its text rows behind the left-over rows
    T_all = []
    for b in range(B):
        t = N_v[b] % n
        K_txt[b, :, t:t + T_own[b]] = p["K_txt"][b, :, :T_own[b]].to(DEV)
        V_txt[b, :, t:t + T_own[b]] = p["V_txt"][b, :, :T_own[b]].to(DEV)
        T_all.append(t + T_own[b])
    T_dev = _i32(T_all)
    ws = kvc.alloc_workspace(layer, B, R_max, T_cap, DEV)
    out = torch.full((B, shape.H_q, 128), float("nan"), dtype=dt, device=DEV)
    kvc.kvc_decode_attend_ragged(layer, p["q"].to(DEV), caps, B, R_max, R_b, K_txt, V_txt, max(T_all), T_dev, T_cap, out, ws)
    torch.cuda.synchronize()
    assert _status(layer, B, R_max, max(T_all), ws) == 0
    want = orc.decode_attend_ragged(tl.np64(p["q"]), K_o, V_o, tl.np64(p["theta"]), tl.np64(p["U"]), tl.np64(p["mu"]),
                                    np.nan_to_num(tl.np64(K_txt)), np.nan_to_num(tl.np64(V_txt)), R_o, T_all, mode)
    tl.assert_close(tl.np64(out), want, dtype, "ragged compress + decode")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])          # three-phase kernels / the resident-parameter kernel
def test_lengths_out_of_range_are_clamped_and_reported(dtype):
    shape = wl.Shape("ragged", 1, 3, 4, 2, 128, 8, 2, 40, 1, dtype, 500)            # n = 64
    p = tl.make_problem(shape, 33, T=40, T_cap=40)
    layer = tl.gpu_layer(shape, p, DEV)
    B, R, n = 3, 2, 64
    caps = caps_full(layer, p, B, R)
    ws = kvc.alloc_workspace(layer, B, R, 40, DEV)
    out = torch.empty((B, 4, 128), dtype=wl.torch_dtype(dtype), device=DEV)
    args = (p["q"].to(DEV), caps, B, R)
    kvc.kvc_decode_attend_ragged(layer, *args, _i32([2, 3, -1]), p["K_txt"].to(DEV), p["V_txt"].to(DEV), 40, _i32([40, 41, 40]),
                                 40, out, ws)
    torch.cuda.synchronize()
    assert _status(layer, B, R, 40, ws) == -8
    K_o, V_o, _ = tl.oracle_run(shape, p)
    want = orc.decode_attend_ragged(tl.np64(p["q"]), K_o, V_o, tl.np64(p["theta"]), tl.np64(p["U"]), tl.np64(p["mu"]),
                                    tl.np64(p["K_txt"]), tl.np64(p["V_txt"]), [2, 2, 0], [40, 40, 40])
    tl.assert_close(tl.np64(out), want, dtype, "clamped lengths")
    kvc.kvc_decode_attend_ragged(layer, *args, _i32([2, 1, 0]), p["K_txt"].to(DEV), p["V_txt"].to(DEV), 40, _i32([40, 0, 7]),
                                 40, out, ws)
    torch.cuda.synchronize()
    assert _status(layer, B, R, 40, ws) == 0             # the next call clears it
    # compress: a run longer than the buffer, more blocks than R_max, more left-over rows than T_cap
    R_b, T_b = _i32([0, 0, 0]), _i32([0, 0, 0])
    tail = torch.empty((B, 2, 5, 128), dtype=wl.torch_dtype(dtype), device=DEV)
    Kv, Vv = p["K_vis"].to(DEV), p["V_vis"].to(DEV)
    for N_v, want_R, want_T in (([129, 64, 0], [2, 1, 0], [0, 0, 0]), ([128, 70, 5], [2, 1, 0], [0, 5, 5])):
        kvc.kvc_compress_ragged(layer, Kv, Vv, B, 2 * n, _i32(N_v), R, caps, tail, tail.clone(), 5, R_b, T_b)
        torch.cuda.synchronize()
        assert kvc.kvc_read_compress_status(layer) == -8
        assert R_b.tolist() == want_R and T_b.tolist() == want_T
    kvc.kvc_compress_ragged(layer, Kv, Vv, B, 2 * n, _i32([128, 69, 5]), R, caps, tail, tail.clone(), 5, R_b, T_b)
    torch.cuda.synchronize()
    assert kvc.kvc_read_compress_status(layer) == 0
    with pytest.raises(kvc.KvcError):
        kvc.kvc_compress_ragged(layer, Kv, Vv, B, 2 * n, None, R, caps, tail, tail, 5, R_b, T_b)
