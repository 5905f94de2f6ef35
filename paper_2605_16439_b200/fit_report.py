"""Accuracy against compression ratio with parameters fitted on the device (synthetic analogue of App. G Table 6 and
App. H Table 7): python -m paper_2605_16439_b200.fit_report [--config 1|2|3] [--out FILE]

For one configuration's block shape (reduced batch and head count) the script
  1. draws training blocks and held-out sequences from the workload generator (smoothed fields; AR(1) frames for video),
  2. fits (U, mu) with kvc_fit_value_pca and theta with kvc_fit_key_reconstructor for every ratio, on the device,
  3. runs kvc_compress + kvc_decode_attend on the held-out sequences in the three modes (both sides, keys only, values
     only) and kvc_attend_full on the uncompressed cache,
  4. prints, per ratio and mode, the mean and minimum cosine similarity of the compressed output to the full-attention
     output over all (sequence, query head) pairs, the fraction of value energy and key energy the fit loses on the
     held-out blocks, and the time the two fits took.
Everything runs through the library's public calls; nothing here is a reference implementation.
"""
from __future__ import annotations

import argparse
import sys
import time

import torch

from . import binding as kvc
from . import build as kvc_build
from . import workloads as wl

RATIOS = (200, 400, 600, 800, 900, 950)
MODES = (("kv", kvc.KVC_MODE_KV), ("k-only", kvc.KVC_MODE_K_ONLY), ("v-only", kvc.KVC_MODE_V_ONLY))


def cosine(a: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    a, b = a.double(), b.double()
    return (a * b).sum(-1) / (a.norm(dim=-1) * b.norm(dim=-1)).clamp_min(1e-300)


def lost_energy(X: torch.Tensor, n: int, rebuild) -> float:
    """sum over blocks || X_blk - rebuild(X_blk) ||^2 / sum || X_blk ||^2 in fp64, X [B, H, R*n, d]."""
    B, H, N, d = X.shape
    blk = X.double().reshape(B, H, N // n, n, d)
    return float(((blk - rebuild(blk)) ** 2).sum() / (blk ** 2).sum())


def run(config: int, q_gain: float, dev: str = "cuda"):
    base = wl.CONFIGS[config]
    H_kv = min(base.H_kv, 2)
    G = base.G
    shape = wl.Shape("fit-report", 1, 4, H_kv * G, H_kv, 128, base.grid, min(base.R, 4), 64, 1, "bf16", 600, base.ar1)
    n, dt = shape.n, torch.bfloat16
    train_K = wl.vision_kv(8, H_kv, 4, shape.grid, 128, 9001, dev, dt, shape.ar1)
    train_V = wl.vision_kv(8, H_kv, 4, shape.grid, 128, 9002, dev, dt, shape.ar1)
    B, R, T = shape.B, shape.R, shape.T0
    K_vis = wl.vision_kv(B, H_kv, R, shape.grid, 128, 9003, dev, dt, shape.ar1)
    V_vis = wl.vision_kv(B, H_kv, R, shape.grid, 128, 9004, dev, dt, shape.ar1)
    K_txt = wl.gaussian((B, H_kv, T, 128), 9005, dev, dt)
    V_txt = wl.gaussian((B, H_kv, T, 128), 9006, dev, dt)
    q = wl.gaussian((B, shape.H_q, 128), 9007, dev, dt, q_gain)

    plain = kvc.Layer(shape.H_q, H_kv, 128, n, 0, dt)
    K_all = torch.cat([K_vis, K_txt], dim=2).contiguous()
    V_all = torch.cat([V_vis, V_txt], dim=2).contiguous()
    S = R * n + T
    full = torch.empty((B, shape.H_q, 128), dtype=dt, device=dev)
    kvc.kvc_attend_full(plain, q, K_all, V_all, B, S, S, full, kvc.alloc_workspace(plain, B, 0, S, dev))
    torch.cuda.synchronize()

    rows = []
    for ratio in RATIOS:
        m = kvc.kvc_retained_len(n, ratio)
        idx = wl.evenly_spaced_idx(n, m)
        t0 = time.perf_counter()
        U, mu, _, sw_v = kvc.kvc_fit_value_pca(train_V, n, m)
        t1 = time.perf_counter()
        theta, sw_k = kvc.kvc_fit_key_reconstructor(train_K, idx, n)
        t2 = time.perf_counter()
        Ud, th = U.double(), theta.double()
        v_lost = lost_energy(V_vis, n, lambda blk: torch.einsum("hjn,bhrjd->bhrnd", Ud, torch.einsum(
            "hjn,bhrnd->bhrjd", Ud, blk - mu.double()[None, :, None, None, :])) + mu.double()[None, :, None, None, :])
        k_lost = lost_energy(K_vis, n, lambda blk: torch.einsum("hjn,bhrjd->bhrnd", th, blk[:, :, :, idx.to(dev).long()]))
        rec = {"ratio": ratio / 1000, "m": m, "v_lost": v_lost, "k_lost": k_lost, "fit_pca_s": t1 - t0, "fit_theta_s": t2 - t1,
               "sweeps": (sw_v, sw_k)}
        for name, mode in MODES:
            layer = kvc.Layer(shape.H_q, H_kv, 128, n, ratio, dt, idx=idx, theta=theta, U=U, mu=mu, mode=mode)
            caps = kvc.alloc_capsules(layer, B, R, dev)
            kvc.kvc_compress(layer, K_vis, V_vis, B, R, caps)
            out = torch.empty_like(full)
            kvc.kvc_decode_attend(layer, q, caps, B, R, K_txt, V_txt, T, T, out, kvc.alloc_workspace(layer, B, R, T, dev))
            torch.cuda.synchronize()
            c = cosine(out, full)
            rec[name] = (float(c.mean()), float(c.min()))
        rows.append(rec)
    return shape, rows


def render(config: int, q_gain: float, shape, rows) -> str:
    out = [f"### config {config} block shape: n = {shape.n}, G = {shape.G}, H_kv = {shape.H_kv}, B = {shape.B}, R = {shape.R}, "
           f"T = {shape.T0}, bf16, query gain {q_gain:g}" + (f", AR(1) {shape.ar1}" if shape.ar1 else ""),
           "",
           "| rho | m | value energy lost | key energy lost | cos kv (mean / min) | cos k-only | cos v-only | fit PCA s (sweeps) | fit theta s (sweeps) |",
           "|---|---|---|---|---|---|---|---|---|"]
    for r in rows:
        out.append(f"| {r['ratio']:.2f} | {r['m']} | {r['v_lost']:.4f} | {r['k_lost']:.4f} | {r['kv'][0]:.4f} / {r['kv'][1]:.4f} | "
                   f"{r['k-only'][0]:.4f} / {r['k-only'][1]:.4f} | {r['v-only'][0]:.4f} / {r['v-only'][1]:.4f} | "
                   f"{r['fit_pca_s']:.2f} ({r['sweeps'][0]}) | {r['fit_theta_s']:.2f} ({r['sweeps'][1]}) |")
    return "\n".join(out) + "\n"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, nargs="*", default=[1, 2, 3])
    ap.add_argument("--q-gain", type=float, nargs="*", default=[1.0, 4.0])
    ap.add_argument("--out", default=None)
    a = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("fit_report needs a CUDA device")
    kvc_build.build()
    text = []
    for c in a.config:
        for g in a.q_gain:
            shape, rows = run(c, g)
            text.append(render(c, g, shape, rows))
            print(text[-1], flush=True)
    if a.out:
        with open(a.out, "w") as f:
            f.write("\n".join(text))


if __name__ == "__main__":
    sys.exit(main())
