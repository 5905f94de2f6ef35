"""Benchmark of the KVCapsule decode hot path on B200: capsule compress + fused reconstruct/decode attention.

One bench "step" is one pass of the whole hot path over one batch of synthetic sequences: every
layer's vision K/V is compressed once (prefill stage), then `decode_steps` decode steps run, each
calling the fused decode attention of every layer with the text tail one row longer than the step
before.  `value` is decode tokens/s of the whole job: sequences x decode steps / time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 1]

Under torchrun (N > 1) every rank runs the same per-GPU batch on its own GPU (weak scaling, no
data-path collective: sequences are independent); time is the max over ranks.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2605_16439_b200 import workloads as wl

FALLBACK_HBM_GBS = 6650.0       # earlier measurement on this machine, used only if MEASURED_PEAKS.json is absent
FALLBACK_BF16_TFLOPS = 1400.0   # sustained dense bf16 of the same earlier measurement
NOMINAL_HBM_GBS = 8000.0        # nominal HBM3e bandwidth: the roofline fraction of the metric is quoted against it

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel from one ncu capture,
# keyed by (kernel, workload name): (bytes, digest of the kernel's source files when the counters were taken).  The
# captures ran at 4 decode steps (text length 130 / 258 / 514; profiles/*.md give the commands); a text row adds exactly
# 2 * B * H_kv * d * 2 bytes, and the figure here is scaled by that amount to the mid-run text length.  For the three-kernel
# path the figure is the sum over its three kernels (one layer call).  When the sources no longer match the digest the
# bench reports traffic = null: the counters belong to another kernel.
KERNEL_SOURCES = {
    "fused": ("kvc_fused.cu", "kvc_fused.cuh", "kvc_tma.cuh", "kvc_async.cuh"),
    "fused_tc": ("kvc_fused_tc.cu", "kvc_fused.cuh", "kvc_tcgen05.cuh", "kvc_tma.cuh", "kvc_async.cuh"),
    "fused_pair": ("kvc_fused_tc.cu", "kvc_fused.cuh", "kvc_tcgen05.cuh", "kvc_tma.cuh", "kvc_async.cuh"),
    "resident": ("kvc_resident.cu", "kvc_resident.cuh", "kvc_tma.cuh", "kvc_async.cuh"),
    "split_scores+split_expand+split_output": ("kvc_split_scores.cu", "kvc_split_expand.cu", "kvc_split_output.cu", "kvc_split.cuh",
                                               "kvc_tcgen05.cuh", "kvc_tma.cuh", "kvc_async.cuh"),
}
NCU_TRAFFIC_BYTES = {
    ("fused", "config1-llava-next-7b"): (208.4e6, "3788d05ac9fe"),
    ("split_scores+split_expand+split_output", "config2-qwen2-vl-7b"): (147.7e6, "b9ec0383c83b"),
    ("resident", "config3-internvl3-8b-video"): (36.0e6, "1e4ede360c43"),
}


def source_digest(kernel: str) -> str:
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES.get(kernel, ()):
        with open(os.path.join(ROOT, "paper_2605_16439_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:12]


def ncu_traffic(kernel: str, workload: str):
    rec = NCU_TRAFFIC_BYTES.get((kernel, workload))
    if rec is None or rec[1] != source_digest(kernel):
        return None
    return rec[0]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", type=int, default=1, help="index into the benchmark configurations (1 = LLaVA-NeXT-7B shape)")
    ap.add_argument("--decode-steps", type=int, default=None, help="override the configuration's decode steps")
    ap.add_argument("--layers", type=int, default=None)
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--ratio", type=int, default=None, help="compression ratio in permille")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-comparator", action="store_true")
    ap.add_argument("--no-profile", action="store_true", help="do not bracket kernels with events in the timed region")
    ap.add_argument("--no-other-configs", dest="other_configs", action="store_false",
                    help="headline configuration only (the default run also times configurations 2 and 3 for two steps each)")
    ap.add_argument("--oracle-decode-steps", type=int, default=96)
    ap.add_argument("--pyramid", type=str, default=None, metavar="LO,HI",
                    help="decode loop with a per-layer ratio rising linearly from LO to HI permille (first to last layer), "
                         "beside the same loop at the uniform mean ratio; one JSON line (not the headline metric)")
    ap.add_argument("--sweep-steps", type=int, default=128, help="decode steps per sweep point (the configuration states 128)")
    ap.add_argument("--sweep", action="store_true",
                    help="configuration 4: ratio x batch x vision tokens on the Qwen2-VL shape; prints one JSON line per point")
    return ap.parse_args()


def pick_shape(a) -> wl.Shape:
    s = wl.CONFIGS[a.config]
    kw = {}
    if a.decode_steps is not None: kw["steps"] = a.decode_steps
    if a.layers is not None: kw["layers"] = a.layers
    if a.batch is not None: kw["B"] = a.batch
    if a.ratio is not None: kw["ratio_permille"] = a.ratio
    return dataclasses.replace(s, **kw)


def elem_bytes(shape) -> int:
    return 2 if shape.dtype == "bf16" else 4


def contract_bytes_per_layer_call(shape, m, T) -> int:
    """Capsule bytes + text-KV bytes + Q/O bytes of one kvc_decode_attend call."""
    b = elem_bytes(shape)
    return (2 * shape.B * shape.H_kv * shape.R * m * shape.d * b + 2 * shape.B * shape.H_kv * T * shape.d * b
            + 2 * shape.B * shape.H_q * shape.d * b)


def stream_kernel_bytes(shape, m, T) -> int:
    """Algorithmic bytes of ONE launch of the scores (or output) kernel: one of K_tilde/V_tilde, one of the
    text K/V, and q (or out)."""
    b = elem_bytes(shape)
    return (shape.B * shape.H_kv * (shape.R * m + T) * shape.d * b + shape.B * shape.H_q * shape.d * b)


# --------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.path = gpu_index, None, None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                c = [x.strip() for x in line.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1])); mx.append(float(c[2]))
                except ValueError:
                    continue
                for nm, v in zip(names, c[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
        os.unlink(self.path)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------- GPU arm
class Job:
    """All device state of one rank's batch: per-layer inputs, parameters, capsule stores, text tails."""

    def __init__(self, shape: wl.Shape, config_index: int, dev, rank: int, ratios=None):
        """ratios: compression ratio in permille per layer (a pyramid schedule); None = the shape's ratio everywhere."""
        from paper_2605_16439_b200 import binding as kvc
        self.kvc, self.shape, self.dev = kvc, shape, dev
        dt = wl.torch_dtype(shape.dtype)
        self.ratios = list(ratios) if ratios is not None else [shape.ratio_permille] * shape.layers
        self.m = kvc.kvc_retained_len(shape.n, shape.ratio_permille)
        self.T_cap = shape.T0 + shape.steps
        self.layers = []
        self.ws = None
        for l, ratio in enumerate(self.ratios):
            seed = wl.layer_seed(config_index, l) + 100000 * rank
            m = kvc.kvc_retained_len(shape.n, ratio)
            p = wl.decode_inputs(shape, m, seed, dev, T=shape.T0, T_cap=self.T_cap)
            if ratio == 0:
                layer = kvc.Layer(shape.H_q, shape.H_kv, shape.d, shape.n, 0, dt, layer=l)
            else:
                layer = kvc.Layer(shape.H_q, shape.H_kv, shape.d, shape.n, ratio, dt, idx=p["idx"],
                                  theta=p["theta"], U=p["U"], mu=p["mu"], layer=l)
            p["layer"], p["m"], p["ratio"] = layer, m, ratio
            p["caps"] = kvc.alloc_capsules(layer, shape.B, shape.R, dev)
            p["out"] = torch.zeros((shape.B, shape.H_q, shape.d), dtype=dt, device=dev)
            self.layers.append(p)
            if ratios is not None or l == 0:       # one workspace serves every layer: the largest request
                ws = kvc.alloc_workspace(layer, shape.B, shape.R, self.T_cap, dev)
                if self.ws is None or ws.numel() * ws.element_size() > self.ws.numel() * self.ws.element_size():
                    self.ws = ws
        self.launches = 0

    def compress_all(self):
        s = self.shape
        for p in self.layers:
            self.kvc.kvc_compress(p["layer"], p["K_vis"], p["V_vis"], s.B, s.R, p["caps"])
        self.launches += sum(0 if r == 0 else 2 for r in self.ratios)

    def decode_step(self, t: int):
        s = self.shape
        T = s.T0 + t
        for p in self.layers:
            self.kvc.kvc_decode_attend(p["layer"], p["q"], p["caps"], s.B, s.R, p["K_txt"], p["V_txt"], T,
                                       self.T_cap, p["out"], self.ws)
        self.launches += len(self.layers)          # lower bound (one-kernel path); the event-bracket pass counts exactly

    def step(self, marks=None):
        """One bench step.  marks: a list that receives (start, after compress, end) events of this step, recorded on the
        launching stream between the library calls (they add no synchronisation)."""
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)] if marks is not None else None
        if ev: ev[0].record()
        self.compress_all()
        if ev: ev[1].record()
        for t in range(self.shape.steps):
            self.decode_step(t)
        if ev:
            ev[2].record()
            marks.append(tuple(ev))


def timed(fn, reps: int, dev) -> float:
    """Milliseconds of `reps` calls of fn on the current stream, device-timed."""
    st, en = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    st.record()
    for _ in range(reps):
        fn()
    en.record()
    torch.cuda.synchronize(dev)
    return st.elapsed_time(en)


def run_e2e(job: Job, dev) -> dict:
    """The same job driven from HOST buffers: per step the vision K/V of every layer, and per decode step the queries
    and the new text K/V rows of all layers, are copied from pinned host memory, and the attention outputs of all
    layers are copied back, all inside the timed region.  The per-decode-step inputs of the layers travel as one packed
    buffer each (queries, key rows, value rows) and the outputs as one: the text tails, queries and outputs of the
    layers are slices of one device tensor each."""
    s, kvc = job.shape, job.kvc
    dt = wl.torch_dtype(s.dtype)
    L = len(job.layers)
    q_all = torch.stack([p["q"] for p in job.layers])                    # [L, B, H_q, d]
    out_all = torch.zeros_like(q_all)
    Kt_all = torch.stack([p["K_txt"] for p in job.layers])               # [L, B, H_kv, T_cap, d]
    Vt_all = torch.stack([p["V_txt"] for p in job.layers])
    for l, p in enumerate(job.layers):                                   # the job's layers now live in the packed tensors
        p["q"], p["out"], p["K_txt"], p["V_txt"] = q_all[l], out_all[l], Kt_all[l], Vt_all[l]
    torch.cuda.empty_cache()
    host_vis = [(p["K_vis"].to("cpu").pin_memory(), p["V_vis"].to("cpu").pin_memory()) for p in job.layers]
    h_q = q_all.to("cpu").pin_memory()
    h_k = Kt_all[:, :, :, 0].contiguous().to("cpu").pin_memory()         # [L, B, H_kv, d]: the row appended per decode step
    h_v = Vt_all[:, :, :, 0].contiguous().to("cpu").pin_memory()
    h_out = torch.empty(out_all.shape, dtype=dt).pin_memory()
    h2d = d2h = 0

    def one_step():
        nonlocal h2d, d2h
        h2d = d2h = 0
        for p, (hk, hv) in zip(job.layers, host_vis):
            p["K_vis"].copy_(hk, non_blocking=True)
            p["V_vis"].copy_(hv, non_blocking=True)
            h2d += hk.numel() * hk.element_size() * 2
            kvc.kvc_compress(p["layer"], p["K_vis"], p["V_vis"], s.B, s.R, p["caps"])
        for t in range(s.steps):
            T = s.T0 + t
            q_all.copy_(h_q, non_blocking=True)
            Kt_all[:, :, :, T - 1].copy_(h_k, non_blocking=True)
            Vt_all[:, :, :, T - 1].copy_(h_v, non_blocking=True)
            for p in job.layers:
                kvc.kvc_decode_attend(p["layer"], p["q"], p["caps"], s.B, s.R, p["K_txt"], p["V_txt"], T, job.T_cap,
                                      p["out"], job.ws)
            h_out.copy_(out_all, non_blocking=True)
            h2d += (h_q.numel() + 2 * h_k.numel()) * h_q.element_size()
            d2h += h_out.numel() * h_out.element_size()

    one_step()                                   # warm-up (also pages the pinned buffers in)
    torch.cuda.synchronize(dev)
    t0 = time.perf_counter()
    ms = timed(one_step, 1, dev)
    wall = (time.perf_counter() - t0) * 1e3
    ms = max(ms, wall)                           # host-side copies and launches count end to end
    return {"ms": ms, "h2d": h2d, "d2h": d2h}


def run_comparator(shape: wl.Shape, dev, reps_layers: int = 8, steps: int = 16) -> dict:
    """Our own uncompressed decode attention (kvc_attend_full) over full vision + text K/V of the same shape."""
    from paper_2605_16439_b200 import binding as kvc
    dt = wl.torch_dtype(shape.dtype)
    S_cap = shape.N_v + shape.T0 + shape.steps
    nl = min(reps_layers, shape.layers)
    layer = kvc.Layer(shape.H_q, shape.H_kv, shape.d, shape.n, 0, dt)
    bufs = []
    for l in range(nl):
        bufs.append((wl.gaussian((shape.B, shape.H_kv, S_cap, shape.d), 900 + l, dev, dt),
                     wl.gaussian((shape.B, shape.H_kv, S_cap, shape.d), 950 + l, dev, dt),
                     wl.gaussian((shape.B, shape.H_q, shape.d), 990 + l, dev, dt)))
    ws = kvc.alloc_workspace(layer, shape.B, 0, S_cap, dev)
    out = torch.empty((shape.B, shape.H_q, shape.d), dtype=dt, device=dev)
    S_mid = shape.N_v + shape.T0 + shape.steps // 2

    def run():
        for _ in range(steps):
            for K, V, q in bufs:
                kvc.kvc_attend_full(layer, q, K, V, shape.B, S_mid, S_cap, out, ws)
    run()
    ms = timed(run, 1, dev)
    per_layer_ms = ms / (steps * nl)
    step_ms = per_layer_ms * shape.layers
    bytes_call = 2 * shape.B * shape.H_kv * S_mid * shape.d * elem_bytes(shape)
    return {"kernel": "kvc_attend_full (uncompressed, our own)", "ms_per_layer_call": per_layer_ms,
            "tokens_per_s": shape.B / (step_ms * 1e-3), "hbm_gbs": bytes_call / (per_layer_ms * 1e-3) / 1e9,
            "kv_len": S_mid, "sample": f"{nl} distinct layers x {steps} calls at the mid-run text length"}


# --------------------------------------------------------------------------------------------- CPU oracle arm
def oracle_sample(shape: wl.Shape, config_index: int, decode_steps: int, budget_s: float = 14.0, threads=None) -> dict:
    """Times the CPU oracle, as it stands, on ONE layer: one compress plus up to `decode_steps` decode steps of
    Algorithm 1's order spread over the run (stopping once `budget_s` seconds of decode work are spent, two steps at
    least), and scales to the full job (layers x steps) by the per-call averages.  threads: limit of the BLAS thread
    pool (None = as the host provides)."""
    import contextlib
    import numpy as np
    from oracle import kvcapsule_oracle as orc
    try:
        from threadpoolctl import threadpool_info, threadpool_limits
        limit = threadpool_limits(limits=threads) if threads else contextlib.nullcontext()
    except Exception:
        threadpool_info, limit = None, contextlib.nullcontext()
    with limit:
        try:
            cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
        except Exception:
            cores = threads or os.cpu_count() or 1
        m = orc.retained_len(shape.n, shape.ratio_permille)
        T_cap = shape.T0 + shape.steps
        p = wl.decode_inputs(shape, m, wl.layer_seed(config_index, 0), "cpu", T=shape.T0, T_cap=T_cap)
        f64 = lambda t: t.float().numpy().astype(np.float64)
        a = {k: f64(p[k]) for k in ("K_vis", "V_vis", "K_txt", "V_txt", "q", "theta", "U", "mu")}
        passthrough = shape.ratio_permille == 0
        t0 = time.perf_counter()
        K_t, V_t = orc.compress(a["K_vis"], a["V_vis"], p["idx"].numpy(), a["U"], a["mu"], shape.n, passthrough)
        t_comp = time.perf_counter() - t0
        ts = []
        stride = max(1, shape.steps // decode_steps)
        picks = list(range(0, shape.steps, stride))[:decode_steps]
        # visit the picked steps from both ends inwards so that a run cut short by the budget still spans the text lengths
        order = [picks[i // 2] if i % 2 == 0 else picks[-1 - i // 2] for i in range(len(picks))]
        for t in order:
            T = shape.T0 + t
            t0 = time.perf_counter()
            orc.decode_attend_fused(a["q"], K_t, V_t, a["theta"], a["U"], a["mu"], a["K_txt"][:, :, :T],
                                    a["V_txt"][:, :, :T], passthrough)
            ts.append(time.perf_counter() - t0)
            if len(ts) >= 2 and sum(ts) >= budget_s:
                break
    t_dec = sum(ts) / len(ts)
    total = shape.layers * (t_comp + shape.steps * t_dec)
    return {"value": shape.B * shape.steps / total, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": (f"1 of {shape.layers} layers, full batch: 1 compress ({t_comp:.2f} s) + {len(ts)} of "
                       f"{shape.steps} decode steps spread over the run ({t_dec * 1e3:.0f} ms each); scaled to "
                       f"layers x steps"),
            "cpu_seconds": t_comp + sum(ts)}


def config_dict(shape: wl.Shape, m: int, extra=None) -> dict:
    c = {"workload": shape.name, "layers": shape.layers, "batch_per_gpu": shape.B, "H_q": shape.H_q,
         "H_kv": shape.H_kv, "d": shape.d, "n": shape.n, "R": shape.R, "m": m,
         "ratio": shape.ratio_permille / 1000.0, "text_tokens": f"{shape.T0}->{shape.T0 + shape.steps}",
         "decode_steps": shape.steps,
         "l2": "inputs larger than L2: every layer call streams its own >126 MB of capsules and text K/V"}
    if extra:
        c.update(extra)
    return c


def run_reference(a, shape, rank):
    if rank != 0:
        return
    from oracle import kvcapsule_oracle as orc
    m = orc.retained_len(shape.n, shape.ratio_permille)
    nd = max(2, a.oracle_decode_steps // 2)
    for _ in range(a.warmup if a.warmup < 2 else 1):
        oracle_sample(shape, a.config, 1)
    vals = [oracle_sample(shape, a.config, nd) for _ in range(a.steps)]
    v = statistics.mean(x["value"] for x in vals)
    line = {"impl": "reference", "metric": "decode tokens/s", "value": v, "unit": "tokens/s", "n_gpus": a.gpus,
            "steps": a.steps, "warmup": a.warmup, "ms_per_step": shape.B * shape.steps / v * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(shape, m),
            "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": vals[0]["cores"], "kind": "oracle",
                             "sample": vals[0]["sample"]},
            "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_sweep(a, dev):
    """Configuration 4 (the sweep): ratio {0,.2,.4,.6,.8} x batch {1,8,32,64} x vision tokens {2048,8192,32768} on the
    Qwen2-VL-7B shape (28 query / 4 KV heads, 32x32 grids), bf16, decode steps of the attention path only.  Two layer
    buffers are rotated (every call still streams more than L2 at the larger points); the uncompressed comparator runs on
    the same KV length.  One JSON line per point."""
    from paper_2605_16439_b200 import binding as kvc
    base = wl.CONFIGS[2]
    dt = torch.bfloat16
    steps, nl = a.sweep_steps, 2
    for nv in (2048, 8192, 32768):
        for B in (1, 8, 32, 64):
            for ratio in (0, 200, 400, 600, 800):
                shape = dataclasses.replace(base, B=B, R=nv // base.n, ratio_permille=ratio, layers=nl, steps=steps)
                m = kvc.kvc_retained_len(shape.n, ratio)
                T0, T_cap = shape.T0, shape.T0 + steps
                layers = []
                for l in range(nl):
                    p = wl.decode_inputs(shape, m, 4000 + l, dev, T=T0, T_cap=T_cap)
                    layer = (kvc.Layer(shape.H_q, shape.H_kv, shape.d, shape.n, 0, dt) if ratio == 0 else
                             kvc.Layer(shape.H_q, shape.H_kv, shape.d, shape.n, ratio, dt, idx=p["idx"], theta=p["theta"],
                                       U=p["U"], mu=p["mu"]))
                    p["layer"] = layer
                    p["caps"] = kvc.alloc_capsules(layer, B, shape.R, dev)
                    kvc.kvc_compress(layer, p["K_vis"], p["V_vis"], B, shape.R, p["caps"])
                    p["out"] = torch.empty((B, shape.H_q, shape.d), dtype=dt, device=dev)
                    if l > 0 or ratio != 0:
                        del p["V_vis"]
                    layers.append(p)
                ws = kvc.alloc_workspace(layers[0]["layer"], B, shape.R, T_cap, dev)

                def run():
                    for t in range(steps):
                        for p in layers:
                            kvc.kvc_decode_attend(p["layer"], p["q"], p["caps"], B, shape.R, p["K_txt"], p["V_txt"], T0 + t,
                                                  T_cap, p["out"], ws)
                run()
                ms = timed(run, 1, dev) / (steps * nl)
                contract = contract_bytes_per_layer_call(shape, m, T0 + (steps - 1) / 2.0)
                # uncompressed comparator over the same sequence length (vision + text rows in one K/V buffer)
                S = nv + T0 + steps // 2
                full = kvc.Layer(shape.H_q, shape.H_kv, shape.d, shape.n, 0, dt)
                Kf = layers[0]["K_vis"].new_empty((B, shape.H_kv, S, shape.d)).normal_()
                Vf = torch.empty_like(Kf).normal_()
                wsf = kvc.alloc_workspace(full, B, 0, S, dev)
                outf = torch.empty((B, shape.H_q, shape.d), dtype=dt, device=dev)
                fn = lambda: [kvc.kvc_attend_full(full, layers[0]["q"], Kf, Vf, B, S, S, outf, wsf) for _ in range(steps)]
                fn()
                ms_full = timed(fn, 1, dev) / steps
                print(json.dumps({"sweep": "config4-qwen2-vl-7b", "vision_tokens": nv, "batch": B, "ratio": ratio / 1000.0, "m": m,
                                  "decode_steps": steps,
                                  "us_per_layer_call": round(ms * 1e3, 2), "tokens_per_s_28_layers": round(B / (ms * 1e-3 * 28), 1),
                                  "contract_gbs": round(contract / (ms * 1e-3) / 1e9, 1),
                                  "frac_of_8tbs": round(contract / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 4),
                                  "uncompressed_us_per_layer_call": round(ms_full * 1e3, 2),
                                  "speedup_vs_uncompressed": round(ms_full / ms, 3)}), flush=True)
                del layers, ws, Kf, Vf, wsf
                torch.cuda.empty_cache()


def run_pyramid(a, shape, dev):
    """Pyramid retention schedule (Sec. 2.4, Sec. 3.2: early layers keep more, deep layers less; the paper prints no
    schedule, so a linear one from LO to HI permille is taken, whose mean is the uniform comparison ratio).  Times the
    decode loop (all layers in model order, every layer its own buffers) once with the schedule and once with the mean
    ratio everywhere, and gives each layer's launch time from events placed between the layers."""
    lo, hi = (int(x) for x in a.pyramid.split(","))
    L = shape.layers
    ratios = [lo + (hi - lo) * l // max(L - 1, 1) for l in range(L)]
    mean = round(sum(ratios) / L)
    out = {"pyramid": shape.name, "schedule": f"linear {lo}..{hi} permille over {L} layers", "mean_ratio_permille": mean,
           "batch": shape.B, "decode_steps": shape.steps}
    for tag, rr in (("pyramid", ratios), ("uniform", [mean] * L)):
        job = Job(dataclasses.replace(shape, ratio_permille=mean), a.config, dev, 0, ratios=rr)
        job.compress_all()
        for p in job.layers:                       # the full-size vision K/V is not needed after compression
            del p["K_vis"], p["V_vis"]
        torch.cuda.empty_cache()
        loop = lambda: [job.decode_step(t) for t in range(shape.steps)]
        loop()
        ms = timed(loop, 1, dev)
        T_mid = shape.T0 + (shape.steps - 1) / 2.0
        contract = sum(contract_bytes_per_layer_call(shape, p["m"], T_mid) for p in job.layers)
        out[tag] = {"ms_per_decode_step": round(ms / shape.steps, 4),
                    "tokens_per_s": round(shape.B * shape.steps / (ms * 1e-3), 1),
                    "contract_gbs": round(contract * shape.steps / (ms * 1e-3) / 1e9, 1),
                    "capsule_mb": round(sum(p["caps"].numel() * p["caps"].element_size() for p in job.layers) / 1e6, 1)}
        if tag == "pyramid":
            # per-layer launch times: events between the layers (the programmatic overlap of consecutive launches is
            # off in this pass, so the sum is a little above the loop time)
            ev = [[torch.cuda.Event(enable_timing=True) for _ in range(L + 1)] for _ in range(shape.steps)]
            s = shape
            torch.cuda.synchronize(dev)
            for t in range(s.steps):
                ev[t][0].record()
                for l, p in enumerate(job.layers):
                    job.kvc.kvc_decode_attend(p["layer"], p["q"], p["caps"], s.B, s.R, p["K_txt"], p["V_txt"], s.T0 + t,
                                              job.T_cap, p["out"], job.ws)
                    ev[t][l + 1].record()
            torch.cuda.synchronize(dev)
            per = []
            for l, p in enumerate(job.layers):
                us = sum(ev[t][l].elapsed_time(ev[t][l + 1]) for t in range(s.steps)) / s.steps * 1e3
                c = contract_bytes_per_layer_call(shape, p["m"], T_mid)
                per.append({"layer": l, "ratio": p["ratio"] / 1000.0, "m": p["m"], "us": round(us, 1),
                            "frac_of_8tbs": round(c / (us * 1e-6) / 1e9 / NOMINAL_HBM_GBS, 3)})
            out["per_layer"] = per
        del job
        torch.cuda.empty_cache()
    out["pyramid_vs_uniform"] = round(out["uniform"]["ms_per_decode_step"] / out["pyramid"]["ms_per_decode_step"], 3)
    print(json.dumps(out))


def load_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm": float(p["hbm_gbs"]), "hbm_src": "measured (MEASURED_PEAKS.json hbm_gbs)",
                "tensor": float(p.get("bf16_tflops_sustained", p.get("bf16_tflops", FALLBACK_BF16_TFLOPS))),
                "tensor_src": "measured (MEASURED_PEAKS.json bf16_tflops_sustained)"}
    return {"hbm": FALLBACK_HBM_GBS, "hbm_src": "fallback", "tensor": FALLBACK_BF16_TFLOPS, "tensor_src": "fallback"}


def measure(shape, config_index, dev, rank, world, local, steps, warmup, profile, peaks, dist=None) -> dict:
    """Warm-up, then `steps` timed bench steps of one configuration on this rank: whole-step time (max over ranks),
    the compress and decode parts of the SAME timed region from events recorded inside it, per-kernel event brackets
    from a second pass, and the roofline objects.  Returns the keys of the JSON line that describe the run (plus the
    job itself under "job")."""
    from paper_2605_16439_b200 import binding as kvc
    job = Job(shape, config_index, dev, rank)
    m = job.m
    for _ in range(warmup):
        job.step()
    torch.cuda.synchronize(dev)
    calls = shape.layers * shape.steps
    job.launches = 0
    sampler = ClockSampler(local)
    if dist is not None:
        dist.barrier()
    sampler.start()
    marks = []
    ms = timed(lambda: job.step(marks), steps, dev)
    clocks = sampler.stop()
    if dist is not None:
        t = torch.tensor([ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.barrier()
        ms = float(t.item())
    ms_compress = sum(e0.elapsed_time(e1) for e0, e1, _ in marks) / steps      # per step, inside the timed region
    ms_decode = sum(e1.elapsed_time(e2) for _, e1, e2 in marks) / steps
    # per-kernel durations: the same steps again with every launch bracketed by two CUDA events on the launching
    # stream (the brackets sit between the kernels, so the programmatic overlap of consecutive kernels is off in this
    # pass and the pass is a little slower than the timed region above)
    prof, ms_bracketed = {}, None
    if profile:
        kvc.kvc_profile_start(steps * (5 * calls + 2 * shape.layers))
        ms_bracketed = timed(job.step, steps, dev) / steps
        kvc.kvc_profile_stop()
        prof = kvc.kvc_profile_read()
        kvc.kvc_profile_start(0)
        kvc.kvc_profile_stop()
        job.launches = int(sum(v[1] for v in prof.values())) // max(steps, 1) * steps
    launches = job.launches

    ms_step = ms / steps
    tokens_per_s = world * shape.B * shape.steps / (ms_step * 1e-3)
    T_mid = shape.T0 + (shape.steps - 1) / 2.0
    contract = contract_bytes_per_layer_call(shape, m, T_mid)
    decode_gbs = contract * calls / (ms_decode * 1e-3) / 1e9
    peak, peak_src = peaks["hbm"], peaks["hbm_src"]

    roofline, kernels = None, {}
    decode_kernels = ("scores", "output", "fused", "fused_tc", "fused_pair", "resident", "split_scores", "split_expand", "split_output")
    if prof:
        tot = sum(v[0] for v in prof.values()) or 1.0
        for k, (t, n) in prof.items():
            if n:
                kernels[k] = {"launches": n, "total_ms": round(t, 3), "avg_us": round(t / n * 1e3, 3),
                              "share": round(t / tot, 4)}
        dom = max(decode_kernels, key=lambda k: prof.get(k, (0.0, 0))[0])
        t_dom, n_dom = prof[dom]
        if dom in ("fused", "fused_tc", "fused_pair", "resident"):
            # one kernel per layer call: its launch duration is the decode part of the timed region over its launches
            # (events recorded inside the timed region, on the launching stream; consecutive launches overlap their
            # prologues, which the per-launch brackets of the second pass forbid)
            alg = contract
            avg_us = ms_decode / calls * 1e3
        elif dom.startswith("split_"):
            # three dependent kernels per layer call that overlap their ramps (programmatic dependent launch): the unit
            # the roofline is taken over is the layer call, against the bytes the whole call must move; per-kernel
            # brackets forbid that overlap and are listed under "kernels" for the shares only
            dom = "split_scores+split_expand+split_output"
            alg = contract
            avg_us = ms_decode / calls * 1e3
            t_dom = sum(prof.get(k, (0.0, 0))[0] for k in ("split_scores", "split_expand", "split_output"))
            n_dom = prof["split_scores"][1]
        else:
            # several kernels per layer call: the dominant one against its own stream (one of K_tilde / V_tilde, the
            # text rows it reads, q or out), from its event brackets
            alg = stream_kernel_bytes(shape, m, T_mid)
            avg_us = t_dom / n_dom * 1e3
        achieved = alg / (avg_us * 1e-6) / 1e9
        roofline = {"kernel": dom, "bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                    "frac": round(achieved / peak, 4), "traffic": ncu_traffic(dom, shape.name), "peak_source": peak_src,
                    "algorithmic_bytes_per_launch": int(alg), "avg_launch_us": round(avg_us, 3),
                    "launches_in_timed_region": calls * steps,
                    "avg_launch_us_bracketed": round(t_dom / n_dom * 1e3, 3)}
    # the prefill-side compress on its own: K and V read in full, capsules written; the value projection is a dense
    # contraction of 2 B H_kv R m n d flop per layer
    b = elem_bytes(shape)
    c_bytes = 2 * shape.B * shape.H_kv * shape.R * shape.n * shape.d * b + 2 * shape.B * shape.H_kv * shape.R * m * shape.d * b
    c_flop = 2.0 * shape.B * shape.H_kv * shape.R * m * shape.n * shape.d
    c_us = ms_compress / shape.layers * 1e3
    compress = {"us_per_layer": round(c_us, 2), "algorithmic_bytes_per_layer": int(c_bytes),
                "achieved_gbs": round(c_bytes / (c_us * 1e-6) / 1e9, 1), "frac_of_hbm_peak": round(c_bytes / (c_us * 1e-6) / 1e9 / peak, 4),
                "flop_per_layer": c_flop, "achieved_tflops": round(c_flop / (c_us * 1e-6) / 1e12, 1),
                "frac_of_tensor_peak": round(c_flop / (c_us * 1e-6) / 1e12 / peaks["tensor"], 4),
                "tensor_peak": peaks["tensor"], "tensor_peak_source": peaks["tensor_src"],
                "bound": "hbm (K and V are read in full; the projection runs on tcgen05 beside the stream)"}
    return {"job": job, "value": round(tokens_per_s, 2), "ms_per_step": round(ms_step, 3),
            "config": config_dict(shape, m), "clocks": clocks, "gpu_launches": launches,
            "ms_per_decode_step": round(ms_decode / shape.steps, 4),
            "ms_per_layer_call": round(ms_decode / calls, 5),
            "ms_compress_all_layers": round(ms_compress, 3),
            "decode_contract_gbs": round(decode_gbs, 1),
            "decode_frac_of_8tbs": round(decode_gbs / NOMINAL_HBM_GBS, 4),
            "decode_frac_of_measured_peak": round(decode_gbs / peak, 4),
            # the same with the parameter bytes (theta, U, mu of the layer: read at least once per layer call, since the
            # parameters of all layers exceed L2) added to the contract bytes
            "decode_full_bytes_frac_of_measured_peak": round(
                (contract + (2 * shape.H_kv * m * shape.n + shape.H_kv * shape.d) * elem_bytes(shape)) * calls
                / (ms_decode * 1e-3) / 1e9 / peak, 4),
            "kernels": kernels, "ms_per_step_bracketed": ms_bracketed, "roofline": roofline, "compress": compress}


def main():
    a = parse_args()
    shape = pick_shape(a)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if a.impl == "reference":
        run_reference(a, shape, rank)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    from paper_2605_16439_b200 import build as kvc_build
    if rank == 0 or not os.path.exists(kvc_build.LIB):
        kvc_build.build()
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    from paper_2605_16439_b200 import binding as kvc

    if a.sweep:
        if rank == 0:
            run_sweep(a, dev)
        return

    if a.pyramid:
        if rank == 0:
            run_pyramid(a, shape, dev)
        return

    peaks = load_peaks()
    res = measure(shape, a.config, dev, rank, world, local, a.steps, max(a.warmup, 3), not a.no_profile, peaks,
                  dist if world > 1 else None)
    job, m = res.pop("job"), res["config"]["m"]
    line = {"metric": "decode tokens/s", "value": res["value"], "unit": "tokens/s", "n_gpus": world,
            "steps": a.steps, "warmup": max(a.warmup, 3), "ms_per_step": res["ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": shape.dtype,
            "data": "synthetic"}
    line.update({k: v for k, v in res.items() if k not in ("value", "ms_per_step")})
    line["config"].update({"global_batch": world * shape.B, "parallelism": f"batch-sharded x{world}"})

    if rank == 0 and world == 1:
        if not a.no_comparator:
            line["comparator"] = run_comparator(shape, dev)
        if not a.no_e2e:
            e = run_e2e(job, dev)
            line["e2e"] = {"value": round(shape.B * shape.steps / (e["ms"] * 1e-3), 2), "unit": "tokens/s",
                           "h2d_bytes_per_step": e["h2d"], "d2h_bytes_per_step": e["d2h"],
                           "ms_per_step": round(e["ms"], 3)}
        if not a.no_cpu_baseline:
            line["cpu_baseline"] = oracle_sample(shape, a.config, a.oracle_decode_steps)
            one = oracle_sample(shape, a.config, 4, budget_s=6.0, threads=1)
            line["cpu_baseline"]["single_thread"] = {"value": one["value"], "unit": "tokens/s", "cores": 1,
                                                     "sample": one["sample"]}
        if a.other_configs and all(x is None for x in (a.layers, a.decode_steps, a.batch, a.ratio)):
            # the other 7B-shaped configurations, a few bench steps each in the same process, each under its own clock
            # sampler: per-layer-call time, roofline and the uncompressed comparator on the same shape
            del job
            torch.cuda.empty_cache()
            line["other_configs"] = []
            for ci in (2, 3):
                if ci == a.config:
                    continue
                oshape = wl.CONFIGS[ci]
                r = measure(oshape, ci, dev, rank, 1, local, 2, 1, not a.no_profile, peaks)
                ojob = r.pop("job")
                del ojob
                torch.cuda.empty_cache()
                comp = run_comparator(oshape, dev) if not a.no_comparator else None
                line["other_configs"].append({
                    "workload": oshape.name, "steps": 2, "warmup": 1, "value": r["value"], "unit": "tokens/s",
                    "ms_per_step": r["ms_per_step"], "us_per_layer_call": round(r["ms_per_layer_call"] * 1e3, 2),
                    "decode_frac_of_measured_peak": r["decode_frac_of_measured_peak"],
                    "decode_frac_of_8tbs": r["decode_frac_of_8tbs"],
                    "decode_full_bytes_frac_of_measured_peak": r["decode_full_bytes_frac_of_measured_peak"],
                    "roofline": r["roofline"], "compress": r["compress"],
                    "kernels": r["kernels"], "config": r["config"], "clocks": r["clocks"],
                    "comparator_us": round(comp["ms_per_layer_call"] * 1e3, 2) if comp else None})
                torch.cuda.empty_cache()
    elif world > 1 and not a.no_e2e:
        e = run_e2e(job, dev)
        t = torch.tensor([e["ms"]], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        line["e2e"] = {"value": round(world * shape.B * shape.steps / (float(t.item()) * 1e-3), 2),
                       "unit": "tokens/s", "h2d_bytes_per_step": e["h2d"], "d2h_bytes_per_step": e["d2h"]}
    line["paper_context"] = "paper: up to 2x decode TPS and 2.4x KV memory at 60% (AMD MI250X, Torch-level); context only"
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
