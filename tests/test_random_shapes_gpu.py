"""Seeded random shapes through the default routing of the library, against the fp64 oracle.

The other GPU tests pick their shapes by hand; here block lengths (square grids from 3 x 3 to 32 x 32), head layouts, batch
sizes, block counts, text lengths, ratios, storage types and one-sided modes are drawn together, so that shape-dependent
choices the library makes (which kernels, how many CTAs per pair, which shared-memory layout) are exercised in combinations
nobody wrote down.  The bound is the contract's (1e-4 for fp32, 2e-2 for bf16 storage) while outputs stay below 2.6 in
magnitude and grows with the magnitude above that, as a bf16 rounding step does.
"""
import random

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


def _bound(dtype, want):
    return tl.TOL[dtype] * max(1.0, float(np.abs(want).max()) / 2.6)


def _shrink(B, R, cost, limit):
    while cost(B, R) > limit and (B > 1 or R > 1):
        if B > 1:
            B = max(1, B // 2)
        else:
            R = max(1, R // 2)
    return B, R


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_uniform_calls_on_random_shapes(seed):
    rng = random.Random(seed)
    paths = set()
    for it in range(24):
        grid = rng.choice([3, 5, 7, 8, 9, 11, 12, 13, 16, 16, 20, 24, 32, 32])
        H_kv = rng.choice([1, 2, 3, 4]); G = rng.choice([1, 2, 3, 4, 7, 8, 9, 16])
        B = rng.choice([1, 2, 3, 5, 8, 19, 40]); R = rng.choice([0, 1, 2, 3, 5])
        B, R = _shrink(B, R, lambda b, r: b * H_kv * G * max(r, 1) * grid ** 4, 2e9)
        T = rng.choice([0, 1, 17, 64, 100, 193, 400])
        if R == 0 and T == 0:
            T = 5
        ratio = rng.choice([0, 200, 400, 600, 600, 800, 900, 950])
        dtype = rng.choice(["bf16", "bf16", "f32"])
        mode = rng.choice(["kv", "kv", "kv", "k", "v"]) if ratio > 0 and R > 0 else "kv"
        shape = wl.Shape("random", 1, B, H_kv * G, H_kv, 128, grid, R, T, 1, dtype, ratio)
        what = f"B={B} H_kv={H_kv} G={G} grid={grid} R={R} T={T} ratio={ratio} {dtype} {mode}"
        p = tl.make_problem(shape, 100 * seed + it, T=T, T_cap=T + rng.choice([0, 3, 8]),
                            recipe=rng.choice(["flat", "peaked", "structured"]))
        _, _, want = tl.oracle_run(shape, p, "fused", mode)
        kvc.kvc_profile_start(64)
        try:
            layer, _, _, out = tl.gpu_run(shape, p, mode=mode)
        finally:
            kvc.kvc_profile_stop()
        paths.add(tuple(k for k, v in kvc.kvc_profile_read().items() if v[1] > 0 and k not in ("gather_keys", "project_values", "usum")))
        kvc.kvc_profile_start(0)
        kvc.kvc_profile_stop()
        got = tl.np64(out)
        assert np.isfinite(got).all(), what
        err = float(np.abs(got - want).max())
        assert err <= _bound(dtype, want), f"{what}: max-abs error {err:.3e}"
    assert len(paths) >= 3          # the draw reaches several of the library's paths


@pytest.mark.parametrize("seed", [21, 22])
def test_ragged_calls_on_random_shapes(seed):
    rng = random.Random(seed)
    i32 = lambda x: torch.tensor(list(x), dtype=torch.int32, device=DEV)
    for it in range(20):
        grid = rng.choice([5, 8, 8, 12, 16, 16, 24, 32])
        H_kv = rng.choice([1, 2, 4]); G = rng.choice([1, 3, 7, 8, 12])
        B = rng.choice([1, 2, 5, 9, 20]); R_max = rng.choice([1, 2, 4, 6])
        B, R_max = _shrink(B, R_max, lambda b, r: b * H_kv * G * r * grid ** 4, 2e9)
        T_cap = rng.choice([1, 40, 130, 300])
        ratio = rng.choice([200, 400, 600, 600, 800, 900])
        dtype = rng.choice(["bf16", "bf16", "f32"]); mode = rng.choice(["kv", "kv", "k", "v"])
        R_b = [rng.randint(0, R_max) for _ in range(B)]
        T_b = [rng.choice([0, 1, T_cap, rng.randint(0, T_cap)]) for _ in range(B)]
        shape = wl.Shape("random-ragged", 1, B, H_kv * G, H_kv, 128, grid, R_max, T_cap, 1, dtype, ratio)
        what = f"B={B} H_kv={H_kv} G={G} grid={grid} R_max={R_max} T_cap={T_cap} ratio={ratio} {dtype} {mode} R_b={R_b} T_b={T_b}"
        p = tl.make_problem(shape, 100 * seed + it, T=T_cap, T_cap=T_cap, recipe=rng.choice(["flat", "peaked"]))
        layer = tl.gpu_layer(shape, p, DEV, mode)
        caps = kvc.alloc_capsules(layer, B, R_max, DEV)
        kvc.kvc_compress(layer, p["K_vis"].to(DEV), p["V_vis"].to(DEV), B, R_max, caps)
        K_g, V_g = kvc.capsule_views(layer, caps, B, R_max)
        K_txt, V_txt = p["K_txt"].to(DEV), p["V_txt"].to(DEV)
        for b in range(B):                      # whatever lies past a sequence's lengths must not be read
            K_g[b, :, R_b[b]:] = float("nan"); V_g[b, :, R_b[b]:] = float("nan")
            K_txt[b, :, T_b[b]:] = float("nan"); V_txt[b, :, T_b[b]:] = float("nan")
        ws = kvc.alloc_workspace(layer, B, R_max, T_cap, DEV)
        ws.fill_(0xFF)
        out = torch.full((B, shape.H_q, 128), float("nan"), dtype=wl.torch_dtype(dtype), device=DEV)
        kvc.kvc_decode_attend_ragged(layer, p["q"].to(DEV), caps, B, R_max, i32(R_b), K_txt, V_txt, max(T_b), i32(T_b), T_cap, out, ws)
        torch.cuda.synchronize()
        assert kvc.kvc_read_device_status(layer, B, R_max, max(T_b), ws) == 0, what
        K_o, V_o = orc.compress(tl.np64(p["K_vis"]), tl.np64(p["V_vis"]), p["idx"].numpy(), tl.np64(p["U"]), tl.np64(p["mu"]),
                                shape.n, False, mode)
        want = orc.decode_attend_ragged(tl.np64(p["q"]), K_o, V_o, tl.np64(p["theta"]), tl.np64(p["U"]), tl.np64(p["mu"]),
                                        tl.np64(p["K_txt"]), tl.np64(p["V_txt"]), R_b, T_b, mode)
        got = tl.np64(out)
        assert np.isfinite(got).all(), what
        err = float(np.abs(got - want).max())
        assert err <= _bound(dtype, want), f"{what}: max-abs error {err:.3e}"
