"""Guard regions around every buffer the library writes: compress, decode (every default path, the ragged and one-sided
calls) and the fits must leave the bytes in front of and behind their outputs, the capsule store and the workspace
untouched.  (A stand-in for a memory checker: it catches stray writes next to the caller's buffers, not reads.)"""
import numpy as np
import pytest
import torch

from paper_2605_16439_b200 import binding as kvc
from paper_2605_16439_b200 import build as kvc_build
from paper_2605_16439_b200 import workloads as wl

import kvc_testlib as tl

pytestmark = pytest.mark.gpu
DEV = "cuda"
GUARD = 4096
PATTERN = 0xA5


@pytest.fixture(scope="module", autouse=True)
def _built():
    kvc_build.build()


class Guarded:
    """A byte buffer with a guard region of GUARD bytes on both sides of a 256-byte aligned payload."""

    def __init__(self, nbytes: int):
        self.n = int(nbytes)
        self.raw = torch.full((self.n + 2 * GUARD + 256,), PATTERN, dtype=torch.uint8, device=DEV)
        self.off = GUARD + (-(self.raw.data_ptr() + GUARD)) % 256
        self.payload = self.raw[self.off:self.off + self.n]

    def view(self, dtype, shape):
        return self.payload.view(dtype).view(shape)

    def intact(self) -> bool:
        return bool((self.raw[:self.off] == PATTERN).all()) and bool((self.raw[self.off + self.n:] == PATTERN).all())


CASES = [  # B, H_q, H_kv, grid, R, T, dtype, mode
    (2, 4, 4, 24, 3, 70, "bf16", "kv"),      # mma.sync one-kernel path (n = 576)
    (2, 14, 2, 32, 3, 130, "bf16", "kv"),    # three-kernel path (n = 1024)
    (3, 14, 2, 16, 5, 77, "bf16", "kv"),     # resident path (n = 256), partials in the workspace
    (2, 8, 2, 12, 2, 33, "f32", "kv"),       # three-phase kernels
    (2, 6, 2, 8, 3, 9, "bf16", "k"),
    (2, 6, 2, 8, 3, 9, "f32", "v"),
    (2, 4, 2, 8, 2, 0, "bf16", "kv"),        # no text
    (38, 2, 2, 32, 1, 0, "bf16", "kv"),      # three-kernel path, one CTA of the output kernel per pair, no text
    (40, 8, 8, 16, 2, 20, "bf16", "kv"),     # resident path, more pairs than SMs
]


@pytest.mark.parametrize("B,H_q,H_kv,grid,R,T,dtype,mode", CASES)
def test_compress_and_decode_write_only_inside_their_buffers(B, H_q, H_kv, grid, R, T, dtype, mode):
    shape = wl.Shape("canary", 1, B, H_q, H_kv, 128, grid, R, T, 1, dtype, 600)
    T_cap = T + 5
    p = tl.make_problem(shape, 77 + grid + R, T=T, T_cap=T_cap, recipe="peaked")
    dt = wl.torch_dtype(dtype)
    layer = tl.gpu_layer(shape, p, DEV, mode)
    caps = Guarded(kvc.kvc_capsule_bytes(layer, B, R))
    ws = Guarded(kvc.kvc_workspace_bytes(layer, B, R, T_cap))
    out = Guarded(B * H_q * 128 * dt.itemsize)
    out_t = out.view(dt, (B, H_q, 128))
    kvc.kvc_compress(layer, p["K_vis"].to(DEV), p["V_vis"].to(DEV), B, R, caps.payload)
    K_txt = p["K_txt"].to(DEV) if T_cap > 0 else None
    V_txt = p["V_txt"].to(DEV) if T_cap > 0 else None
    for _ in range(2):                                   # the second call reads the settled store early
        kvc.kvc_decode_attend(layer, p["q"].to(DEV), caps.payload, B, R, K_txt, V_txt, T, T_cap, out_t, ws.payload)
    torch.cuda.synchronize()
    assert caps.intact() and ws.intact() and out.intact()
    assert kvc.kvc_read_device_status(layer, B, R, T, ws.payload) == 0
    _, _, want = tl.oracle_run(shape, p, "fused", mode)
    tl.assert_close(tl.np64(out_t), want, dtype, "guarded buffers")
    # per-sequence lengths on the same guarded buffers
    R_b = torch.tensor([R] + [max(R - 1, 0)] * (B - 1), dtype=torch.int32, device=DEV)
    T_b = torch.tensor([T] + [T // 2] * (B - 1), dtype=torch.int32, device=DEV)
    kvc.kvc_decode_attend_ragged(layer, p["q"].to(DEV), caps.payload, B, R, R_b, K_txt, V_txt, T, T_b, T_cap, out_t, ws.payload)
    torch.cuda.synchronize()
    assert caps.intact() and ws.intact() and out.intact()


def test_ragged_compress_and_fits_write_only_inside_their_buffers():
    n, R_max, T_cap, B, H = 64, 3, 70, 3, 2
    shape = wl.Shape("canary", 1, B, 4, H, 128, 8, 4, T_cap, 1, "bf16", 600)
    p = tl.make_problem(shape, 5150, T=T_cap, T_cap=T_cap)
    layer = tl.gpu_layer(shape, p, DEV)
    caps = Guarded(kvc.kvc_capsule_bytes(layer, B, R_max))
    kt, vt = Guarded(B * H * T_cap * 256), Guarded(B * H * T_cap * 256)
    rb, tb = Guarded(B * 4), Guarded(B * 4)
    N_v = torch.tensor([0, 3 * n, 2 * n + 63], dtype=torch.int32, device=DEV)
    kvc.kvc_compress_ragged(layer, p["K_vis"].to(DEV), p["V_vis"].to(DEV), B, 4 * n, N_v, R_max, caps.payload,
                            kt.view(torch.bfloat16, (B, H, T_cap, 128)), vt.view(torch.bfloat16, (B, H, T_cap, 128)), T_cap,
                            rb.view(torch.int32, (B,)), tb.view(torch.int32, (B,)))
    torch.cuda.synchronize()
    assert kvc.kvc_read_compress_status(layer) == 0
    assert rb.view(torch.int32, (B,)).tolist() == [0, 3, 2] and tb.view(torch.int32, (B,)).tolist() == [0, 0, 63]
    assert all(g.intact() for g in (caps, kt, vt, rb, tb))
    # the fits: outputs and workspace
    m = layer.m
    lib = kvc._lib()
    U, mu, th = Guarded(H * m * n * 2), Guarded(H * 128 * 2), Guarded(H * m * n * 2)
    eig, fws = Guarded(H * n * 8), Guarded(lib.kvc_fit_workspace_bytes(H, n))
    V = p["V_vis"].to(DEV).contiguous()
    assert lib.kvc_fit_value_pca(V.data_ptr(), B, 4, H, n, m, 1, U.payload.data_ptr(), mu.payload.data_ptr(),
                                 eig.payload.data_ptr(), fws.payload.data_ptr(), None, None) == 0
    idx = p["idx"].to(torch.int32).contiguous()
    import ctypes as C
    assert lib.kvc_fit_key_reconstructor(V.data_ptr(), B, 4, H, n, m, C.cast(idx.data_ptr(), C.POINTER(C.c_int32)), 0, 1e-10, 1,
                                         th.payload.data_ptr(), fws.payload.data_ptr(), None, None) == 0
    torch.cuda.synchronize()
    assert all(g.intact() for g in (U, mu, th, eig, fws))
    assert torch.isfinite(U.view(torch.bfloat16, (H, m, n)).float()).all()
