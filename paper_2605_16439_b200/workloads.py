"""Seeded synthetic inputs for the KVCapsule decode path.

This module only draws random tensors; it holds none of the method's arithmetic
(the retained length m is passed in by the caller).  The same generated buffers
are handed to the CPU oracle and to the CUDA library, so neither depends on the
other.  Everything is produced with torch ops so that the benchmark can draw
full-size workloads directly in device memory; parity tests draw on the CPU.

Recipe (stands in for the vision/text activations of LLaVA-NeXT / Qwen2-VL /
InternVL3-shaped models, which are not available offline):
  * vision K and V, independently per (sequence, KV head, block, channel):
    N(0,1) field on the block's g x g patch grid, 3x3 box filter over the grid
    (mean over the in-grid neighbours at the border), plus 0.1 * N(0,1) noise;
    tokens in row-major grid order.
  * video: consecutive blocks are frames of an AR(1) process with coefficient
    rho_t: x_0 = e_0, x_f = rho_t x_{f-1} + sqrt(1 - rho_t^2) e_f, each e_f a
    smoothed field as above.
  * text K/V and the decode query: N(0,1).
  * parameters theta, U [H_kv,m,n] and mu [H_kv,d]: N(0, 1/d) (recipe "flat": near-uniform softmaxes).
  * recipe "peaked": theta ~ N(0, 75/m) instead, which gives the expanded vision logits a standard
    deviation of about 3 on the smoothed fields (a few positions dominate every softmax); text keys
    ~ N(0, 3.5^2) so that the text logits are as peaked and both sides carry probability mass.
  * recipe "structured": theta[j, i] = 1 where idx[j] is the retained position nearest to i (every
    position copies the score of its nearest retained key; theta[:, idx] = I), U with orthonormal
    rows (QR of a Gaussian matrix), the query scaled by 8 (logit standard deviation about 3) and the
    text keys ~ N(0, 0.45^2) (the scale of the smoothed vision keys, so text logits are alike).
    Both sharp recipes scale the vision and text values (by 0.4 and 0.75) so that the outputs, which
    are close to single value rows there, stay below about 2.6 in magnitude: one bf16 step is 2^-7
    of the magnitude, and the absolute parity bound of the bf16 path is stated for outputs of order 1.
  * retained indices: evenly spaced, idx[j] = floor(j n / m); or a sorted seeded
    random subset (irregular gathers).
bf16 workloads are rounded to bf16 once, here, and both sides start from the
rounded values.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Shape:
    """One workload shape (paper notation)."""
    name: str
    layers: int
    B: int
    H_q: int
    H_kv: int
    d: int
    grid: int          # g: block = g x g patch grid, n = g*g
    R: int             # vision blocks per sequence
    T0: int            # text tokens at the first decode step
    steps: int         # decode steps
    dtype: str         # "f32" | "bf16"
    ratio_permille: int = 600
    ar1: float = 0.0   # temporal AR(1) coefficient across blocks (video)

    @property
    def n(self) -> int:
        return self.grid * self.grid

    @property
    def G(self) -> int:
        return self.H_q // self.H_kv

    @property
    def N_v(self) -> int:
        return self.R * self.n


# The five benchmark configurations (index = config number).
CONFIGS = (
    Shape("config0-single-layer-fp32", 1, 1, 8, 2, 128, 24, 1, 32, 1, "f32"),
    Shape("config1-llava-next-7b", 32, 8, 32, 32, 128, 24, 5, 128, 256, "bf16"),
    Shape("config2-qwen2-vl-7b", 28, 16, 28, 4, 128, 32, 8, 256, 512, "bf16"),
    Shape("config3-internvl3-8b-video", 28, 4, 28, 4, 128, 16, 32, 512, 1024, "bf16", ar1=0.9),
)


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def smoothed_field(lead: tuple, grid: int, d: int, gen: torch.Generator, device) -> torch.Tensor:
    """[*lead, grid*grid, d] fp32: box-filtered Gaussian field per channel plus 0.1 noise."""
    n = grid * grid
    numel_lead = int(math.prod(lead)) if lead else 1
    base = torch.randn((numel_lead * d, 1, grid, grid), generator=gen, device=device, dtype=torch.float32)
    sm = torch.nn.functional.avg_pool2d(base, 3, stride=1, padding=1, count_include_pad=False)
    del base
    sm = sm.reshape(numel_lead, d, n).transpose(1, 2)          # token-major, channel-minor
    noise = torch.randn((numel_lead, n, d), generator=gen, device=device, dtype=torch.float32)
    out = sm + 0.1 * noise
    return out.reshape(*lead, n, d).contiguous()


def vision_kv(B: int, H_kv: int, R: int, grid: int, d: int, seed: int, device="cpu",
              dtype=torch.float32, ar1: float = 0.0) -> torch.Tensor:
    """One of K_vis / V_vis: [B, H_kv, R*n, d]."""
    gen = _gen(seed, device)
    n = grid * grid
    if ar1 == 0.0:
        x = smoothed_field((B, H_kv, R), grid, d, gen, device)
    else:
        x = torch.empty((B, H_kv, R, n, d), device=device, dtype=torch.float32)
        prev = None
        for f in range(R):
            e = smoothed_field((B, H_kv), grid, d, gen, device)
            prev = e if prev is None else ar1 * prev + math.sqrt(1.0 - ar1 * ar1) * e
            x[:, :, f] = prev
    return x.reshape(B, H_kv, R * n, d).to(dtype).contiguous()


def gaussian(shape: tuple, seed: int, device="cpu", dtype=torch.float32, std: float = 1.0) -> torch.Tensor:
    gen = _gen(seed, device)
    return (torch.randn(shape, generator=gen, device=device, dtype=torch.float32) * std).to(dtype).contiguous()


def params(H_kv: int, m: int, n: int, d: int, seed: int, device="cpu", dtype=torch.float32):
    """(theta, U, mu) ~ N(0, 1/d) in the shapes of App. D."""
    std = 1.0 / math.sqrt(d)
    theta = gaussian((H_kv, m, n), seed * 7 + 1, device, dtype, std)
    U = gaussian((H_kv, m, n), seed * 7 + 2, device, dtype, std)
    mu = gaussian((H_kv, d), seed * 7 + 3, device, dtype, std)
    return theta, U, mu


def peaked_params(H_kv: int, m: int, n: int, d: int, seed: int, device="cpu", dtype=torch.float32):
    """Recipe "peaked": as `params`, with theta ~ N(0, 75/m)."""
    theta = gaussian((H_kv, m, n), seed * 7 + 1, device, dtype, math.sqrt(75.0 / m))
    U = gaussian((H_kv, m, n), seed * 7 + 2, device, dtype, 1.0 / math.sqrt(d))
    mu = gaussian((H_kv, d), seed * 7 + 3, device, dtype, 1.0 / math.sqrt(d))
    return theta, U, mu


def structured_params(H_kv: int, m: int, n: int, d: int, idx: torch.Tensor, seed: int, device="cpu",
                      dtype=torch.float32):
    """Recipe "structured": nearest-retained-position one-hot theta, orthonormal rows in U, Gaussian mu."""
    idx2 = idx.to(torch.int64).reshape(-1, m)                       # [1 or H_kv, m]
    pos = torch.arange(n, dtype=torch.int64)
    theta = torch.zeros((H_kv, m, n), dtype=torch.float32)
    for h in range(H_kv):
        ih = idx2[h if idx2.shape[0] > 1 else 0]
        nearest = torch.argmin((pos[None, :] - ih[:, None]).abs(), dim=0)   # [n] -> row j of the nearest retained key
        theta[h, nearest, pos] = 1.0
    gen = _gen(seed * 7 + 2, "cpu")
    U = torch.stack([torch.linalg.qr(torch.randn((n, m), generator=gen, dtype=torch.float64))[0].T for _ in range(H_kv)])
    mu = gaussian((H_kv, d), seed * 7 + 3, "cpu", torch.float32, 1.0 / math.sqrt(d))
    return (theta.to(dtype).to(device).contiguous(), U.to(torch.float32).to(dtype).to(device).contiguous(),
            mu.to(dtype).to(device).contiguous())


def evenly_spaced_idx(n: int, m: int) -> torch.Tensor:
    """idx[j] = floor(j n / m), strictly increasing for m <= n; int32 [m]."""
    j = torch.arange(m, dtype=torch.int64)
    return ((j * n) // m).to(torch.int32)


def random_sorted_idx(n: int, m: int, seed: int, H_kv: int = 0) -> torch.Tensor:
    """Sorted random m-subset of 0..n-1; [m] if H_kv == 0 else one subset per KV head [H_kv, m]."""
    gen = _gen(seed, "cpu")
    rows = max(H_kv, 1)
    out = torch.stack([torch.sort(torch.randperm(n, generator=gen)[:m]).values for _ in range(rows)])
    out = out.to(torch.int32)
    return out if H_kv else out[0]


def layer_seed(config_index: int, layer: int) -> int:
    return 1000 * config_index + layer


def decode_inputs(shape: Shape, m: int, seed: int, device="cpu", T: int | None = None,
                  T_cap: int | None = None, recipe: str = "flat", idx: torch.Tensor | None = None):
    """All tensors of one layer's decode problem, in the storage dtype of `shape`.

    Returns a dict: K_vis, V_vis [B,H_kv,N_v,d]; K_txt, V_txt [B,H_kv,T_cap,d] (rows >= T are
    filled too, they must not influence the result); q [B,H_q,d]; theta, U, mu; idx [m].
    recipe: "flat" (the benchmark configurations), "peaked" or "structured" (module docstring); idx: the retained
    index set to use instead of the evenly spaced one.
    """
    dt = torch_dtype(shape.dtype)
    T = shape.T0 if T is None else T
    T_cap = T if T_cap is None else T_cap
    s = seed * 16
    idx = evenly_spaced_idx(shape.n, m) if idx is None else idx
    q_gain, kt_gain, v_gain = 1.0, 1.0, 1.0      # v_gain keeps the sharp recipes' outputs within |y| < 2.6 (one bf16 step there: 2^-7)
    if recipe == "flat":
        theta, U, mu = params(shape.H_kv, m, shape.n, shape.d, s + 5, device, dt)
    elif recipe == "peaked":
        theta, U, mu = peaked_params(shape.H_kv, m, shape.n, shape.d, s + 5, device, dt)
        kt_gain, v_gain = 3.5, 0.4
    elif recipe == "structured":
        theta, U, mu = structured_params(shape.H_kv, m, shape.n, shape.d, idx, s + 5, device, dt)
        q_gain, kt_gain, v_gain = 8.0, 0.45, 0.75
    else:
        raise ValueError(f"unknown recipe {recipe!r}")
    if v_gain != 1.0:
        mu = _scaled(mu.float(), v_gain, dt)           # the centring vector lives on the values' scale
    return dict(
        K_vis=vision_kv(shape.B, shape.H_kv, shape.R, shape.grid, shape.d, s + 0, device, dt, shape.ar1),
        V_vis=_scaled(vision_kv(shape.B, shape.H_kv, shape.R, shape.grid, shape.d, s + 1, device, torch.float32, shape.ar1), v_gain, dt),
        K_txt=gaussian((shape.B, shape.H_kv, T_cap, shape.d), s + 2, device, dt, kt_gain),
        V_txt=gaussian((shape.B, shape.H_kv, T_cap, shape.d), s + 3, device, dt, v_gain),
        q=gaussian((shape.B, shape.H_q, shape.d), s + 4, device, dt, q_gain),
        theta=theta, U=U, mu=mu,
        idx=idx,
        T=T, T_cap=T_cap,
    )


def _scaled(x: torch.Tensor, gain: float, dtype) -> torch.Tensor:
    return (x if gain == 1.0 else x * gain).to(dtype).contiguous()


def shard_batch(B_total: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous slice [lo, hi) of the sequences owned by `rank` (no data-path exchange)."""
    base, rem = divmod(B_total, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)
