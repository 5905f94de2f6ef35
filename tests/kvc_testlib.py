"""Shared helpers of the parity tests: run the CUDA path and the CPU oracle on the same buffers."""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from oracle import kvcapsule_oracle as orc
from paper_2605_16439_b200 import binding as kvc
from paper_2605_16439_b200 import workloads as wl

TOL = {"f32": 1e-4, "bf16": 2e-2}       # max-abs bounds per storage type (fp32 accumulation in both): the contract

# Regression bounds, asserted beside the contract: the kernels sit well inside it, and a test that only checked the
# contract could not tell a wrong block order from rounding.  bf16: the output carries one rounding (2^-9 relative) on
# top of the roundings of the stored scores, probabilities and weights; the absolute floor covers outputs near zero.
REG_REL = {"f32": 5e-6, "bf16": 1.5e-2}      # observed on B200: at most 1.5e-6 (fp32) and 9.3e-3 (bf16) of max|out|; the bf16 maximum is
                                             # the same to four digits for two unrelated kernels: the rounding of the stored capsules sets it
REG_ABS = {"f32": 5e-6, "bf16": 3.0e-3}


def regression_bound(dtype: str, out_max: float) -> float:
    """max-abs error a correct kernel stays below on an output whose largest magnitude is out_max."""
    return min(TOL[dtype], max(REG_ABS[dtype] * min(1.0, 4.0 * out_max), REG_REL[dtype] * out_max))


# the reduced shapes of the 7B-shaped configurations that the parity tests run (config index, overrides)
REDUCED_7B = [
    (1, dict(B=2, H_q=4, H_kv=4)),              # LLaVA-NeXT shape: MHA, n=576, m=231, R=5
    (2, dict(B=2, H_q=14, H_kv=2, R=3)),        # Qwen2-VL shape: G=7, n=1024, m=410
    (3, dict(B=1, H_q=7, H_kv=1, R=6)),         # InternVL3 video shape: n=256, m=103, AR(1) frames
]
RECIPES = ("flat", "peaked", "structured")


def assert_close(got: np.ndarray, want: np.ndarray, dtype: str, what: str = "") -> float:
    """Contract bound and regression bound on one output; returns the max-abs error."""
    assert np.isfinite(got).all(), what
    err = float(np.abs(got - want).max())
    assert err <= TOL[dtype], f"{what} max-abs error {err} > contract {TOL[dtype]}"
    reg = regression_bound(dtype, float(np.abs(want).max()))
    assert err <= reg, f"{what} max-abs error {err} within the contract but above the regression bound {reg}"
    return err


def np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy().astype(np.float64)


def make_problem(shape: wl.Shape, seed: int, T=None, T_cap=None, idx=None, recipe="flat"):
    m = orc.retained_len(shape.n, shape.ratio_permille)
    p = wl.decode_inputs(shape, m, seed, "cpu", T, T_cap, recipe=recipe, idx=idx)
    p["m"] = m
    return p


MODES = {"kv": kvc.KVC_MODE_KV, "k": kvc.KVC_MODE_K_ONLY, "v": kvc.KVC_MODE_V_ONLY}


def oracle_run(shape: wl.Shape, p, form: str = "fused", mode: str = "kv"):
    """(K_tilde, V_tilde, out) in fp64 from the (already rounded) storage-dtype inputs."""
    passthrough = shape.ratio_permille == 0
    T = p["T"]
    args = [np64(p[k]) for k in ("K_vis", "V_vis")]
    K_t, V_t = orc.compress(args[0], args[1], p["idx"].numpy(), np64(p["U"]), np64(p["mu"]), shape.n, passthrough, mode)
    f = orc.decode_attend_fused if form == "fused" else orc.decode_attend_definition
    out = f(np64(p["q"]), K_t, V_t, np64(p["theta"]), np64(p["U"]), np64(p["mu"]),
            np64(p["K_txt"])[:, :, :T], np64(p["V_txt"])[:, :, :T], passthrough, mode)
    return K_t, V_t, out


def gpu_layer(shape: wl.Shape, p, dev="cuda", mode: str = "kv"):
    dt = wl.torch_dtype(shape.dtype)
    if shape.ratio_permille == 0:
        return kvc.Layer(shape.H_q, shape.H_kv, shape.d, shape.n, 0, dt)
    # a one-sided mode gets only the parameters of the side it compresses
    return kvc.Layer(shape.H_q, shape.H_kv, shape.d, shape.n, shape.ratio_permille, dt,
                     idx=p["idx"] if mode != "v" else None, theta=p["theta"].to(dev) if mode != "v" else None,
                     U=p["U"].to(dev) if mode != "k" else None, mu=p["mu"].to(dev) if mode != "k" else None,
                     mode=MODES[mode])


def gpu_run(shape: wl.Shape, p, dev="cuda", mode: str = "kv"):
    """(K_tilde, V_tilde, out) from the CUDA library through the C ABI."""
    layer = gpu_layer(shape, p, dev, mode)
    B, R, T, T_cap = shape.B, shape.R, p["T"], p["T_cap"]
    caps = kvc.alloc_capsules(layer, B, R, dev)
    kvc.kvc_compress(layer, p["K_vis"].to(dev), p["V_vis"].to(dev), B, R, caps)
    ws = kvc.alloc_workspace(layer, B, R, T_cap, dev)
    out = torch.full((B, shape.H_q, shape.d), float("nan"), dtype=wl.torch_dtype(shape.dtype), device=dev)
    K_txt = p["K_txt"].to(dev) if T_cap > 0 else None
    V_txt = p["V_txt"].to(dev) if T_cap > 0 else None
    kvc.kvc_decode_attend(layer, p["q"].to(dev), caps if R > 0 else None, B, R, K_txt, V_txt, T, T_cap, out, ws)
    torch.cuda.synchronize()
    K_t, V_t = kvc.capsule_views(layer, caps, B, R) if R > 0 else (None, None)
    return layer, K_t, V_t, out


def small(shape: wl.Shape, **kw) -> wl.Shape:
    return dataclasses.replace(shape, **kw)
