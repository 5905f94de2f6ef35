"""Thin ctypes binding of libkvc.so: argument marshalling only, every step runs in the CUDA kernels.

Function names mirror the C ABI declared in include/kvc.h.  torch is used for device memory and
the current stream; there is no CPU fallback: a missing library or a failing call raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libkvc.so")

KVC_F32, KVC_BF16 = 0, 1
_DTYPES = {torch.float32: KVC_F32, torch.bfloat16: KVC_BF16}


class KvcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib().kvc_strerror(status).decode() if _LIB is not None else "?"
        if status == -6 and _LIB is not None:
            msg += ": " + _lib().kvc_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} (status {status})")


class kvc_layer_desc(C.Structure):
    _fields_ = [("layer", C.c_int), ("H_q", C.c_int), ("H_kv", C.c_int), ("d", C.c_int), ("n", C.c_int),
                ("ratio_permille", C.c_int), ("dtype", C.c_int), ("idx", C.POINTER(C.c_int32)),
                ("idx_per_head", C.c_int), ("theta", C.c_void_p), ("U", C.c_void_p), ("mu", C.c_void_p),
                ("mode", C.c_int)]


KVC_MODE_KV, KVC_MODE_K_ONLY, KVC_MODE_V_ONLY = 0, 1, 2


_LIB = None


def _lib() -> C.CDLL:
    """Loads libkvc.so once; raises if it has not been built (python -m paper_2605_16439_b200.build)."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_16439_b200.build`")
        lib = C.CDLL(LIB_PATH)
        vp, i = C.c_void_p, C.c_int
        lib.kvc_retained_len.argtypes = [i, i]; lib.kvc_retained_len.restype = i
        lib.kvc_layer_create.argtypes = [C.POINTER(kvc_layer_desc), C.POINTER(vp)]; lib.kvc_layer_create.restype = i
        lib.kvc_layer_destroy.argtypes = [vp]; lib.kvc_layer_destroy.restype = i
        lib.kvc_layer_m.argtypes = [vp]; lib.kvc_layer_m.restype = i
        lib.kvc_layer_capsules_written.argtypes = [vp]; lib.kvc_layer_capsules_written.restype = i
        lib.kvc_layer_rows.argtypes = [vp, C.POINTER(i), C.POINTER(i)]; lib.kvc_layer_rows.restype = i
        lib.kvc_capsule_bytes.argtypes = [vp, i, i]; lib.kvc_capsule_bytes.restype = C.c_size_t
        lib.kvc_workspace_bytes.argtypes = [vp, i, i, i]; lib.kvc_workspace_bytes.restype = C.c_size_t
        lib.kvc_compress.argtypes = [vp, vp, vp, i, i, vp, vp]; lib.kvc_compress.restype = i
        lib.kvc_decode_attend.argtypes = [vp, vp, vp, i, i, vp, vp, i, i, vp, vp, vp]
        lib.kvc_decode_attend.restype = i
        lib.kvc_compress_ragged.argtypes = [vp, vp, vp, i, i, vp, i, vp, vp, vp, i, vp, vp, vp]
        lib.kvc_compress_ragged.restype = i
        lib.kvc_decode_attend_ragged.argtypes = [vp, vp, vp, i, i, vp, vp, vp, i, vp, i, vp, vp, vp]
        lib.kvc_decode_attend_ragged.restype = i
        lib.kvc_fit_workspace_bytes.argtypes = [i, i]; lib.kvc_fit_workspace_bytes.restype = C.c_size_t
        lib.kvc_fit_value_pca.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, vp, vp, C.POINTER(i)]
        lib.kvc_fit_value_pca.restype = i
        lib.kvc_fit_key_reconstructor.argtypes = [vp, i, i, i, i, i, C.POINTER(C.c_int32), i, C.c_double, i, vp, vp, vp,
                                                  C.POINTER(i)]
        lib.kvc_fit_key_reconstructor.restype = i
        lib.kvc_attend_full.argtypes = [vp, vp, vp, vp, i, i, i, vp, vp, vp]; lib.kvc_attend_full.restype = i
        lib.kvc_decode_attend_static.argtypes = [vp, vp, vp, i, i, vp, vp, i, i, vp, vp]
        lib.kvc_decode_attend_static.restype = i
        lib.kvc_static_scratch_bytes.argtypes = []; lib.kvc_static_scratch_bytes.restype = C.c_size_t
        lib.kvc_read_device_status.argtypes = [vp, i, i, i, vp, C.POINTER(i)]
        lib.kvc_read_device_status.restype = i
        lib.kvc_read_compress_status.argtypes = [vp, C.POINTER(i)]; lib.kvc_read_compress_status.restype = i
        lib.kvc_selftest_bounded_wait.argtypes = [vp]; lib.kvc_selftest_bounded_wait.restype = i
        lib.kvc_collapse_theta.argtypes = [vp, vp, i, i, i, i, i, vp, vp]; lib.kvc_collapse_theta.restype = i
        lib.kvc_export_maps.argtypes = [vp, i, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        lib.kvc_export_maps.restype = i
        lib.kvc_strerror.argtypes = [i]; lib.kvc_strerror.restype = C.c_char_p
        lib.kvc_last_cuda_error.argtypes = []; lib.kvc_last_cuda_error.restype = C.c_char_p
        lib.kvc_profile_start.argtypes = [i]; lib.kvc_profile_start.restype = i
        lib.kvc_profile_stop.argtypes = []; lib.kvc_profile_stop.restype = i
        lib.kvc_profile_read.argtypes = [i, C.POINTER(C.c_double), C.POINTER(C.c_longlong)]
        lib.kvc_profile_read.restype = i
        lib.kvc_kernel_name.argtypes = [i]; lib.kvc_kernel_name.restype = C.c_char_p
        _LIB = lib
    return _LIB


def _check(status: int, where: str) -> None:
    if status != 0:
        raise KvcError(status, where)


def _ptr(t) -> int | None:
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensors passed to the kvc library must be contiguous")
    return t.data_ptr()


def _stream(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def kvc_retained_len(n: int, ratio_permille: int) -> int:
    return _lib().kvc_retained_len(n, ratio_permille)


class Layer:
    """Owns one kvc_layer handle and keeps the borrowed parameter tensors alive."""

    def __init__(self, H_q: int, H_kv: int, d: int, n: int, ratio_permille: int, dtype: torch.dtype,
                 idx=None, theta=None, U=None, mu=None, layer: int = 0, mode: int = KVC_MODE_KV):
        if dtype not in _DTYPES:
            raise KvcError(-3, "kvc_layer_create") if _LIB else ValueError("unsupported dtype")
        self.H_q, self.H_kv, self.d, self.n, self.dtype = H_q, H_kv, d, n, dtype
        self.ratio_permille = ratio_permille
        self._keep = (theta, U, mu)
        desc = kvc_layer_desc()
        desc.layer, desc.H_q, desc.H_kv, desc.d, desc.n = layer, H_q, H_kv, d, n
        desc.ratio_permille, desc.dtype = ratio_permille, _DTYPES[dtype]
        desc.mode = mode
        idx_host = None
        if idx is not None:
            idx_host = idx.detach().to("cpu", torch.int32).contiguous()
            desc.idx = C.cast(idx_host.data_ptr(), C.POINTER(C.c_int32))
            desc.idx_per_head = 1 if idx_host.dim() == 2 else 0
        for name, t in (("theta", theta), ("U", U), ("mu", mu)):
            if t is not None and t.dtype != dtype:
                raise ValueError(f"{name} must have the layer's storage dtype")
            setattr(desc, name, _ptr(t))
        h = C.c_void_p()
        _check(_lib().kvc_layer_create(C.byref(desc), C.byref(h)), "kvc_layer_create")
        self.handle = h
        self.m = _lib().kvc_layer_m(h)
        mk, mv = C.c_int(), C.c_int()
        _check(_lib().kvc_layer_rows(h, C.byref(mk), C.byref(mv)), "kvc_layer_rows")
        self.m_k, self.m_v = mk.value, mv.value

    def close(self):
        if getattr(self, "handle", None) and _LIB is not None:      # at interpreter exit the library may be gone already
            try:
                _LIB.kvc_layer_destroy(self.handle)
            except Exception:
                pass
            self.handle = None

    __del__ = close


def kvc_capsule_bytes(layer: Layer, B: int, R: int) -> int:
    return _lib().kvc_capsule_bytes(layer.handle, B, R)


def kvc_workspace_bytes(layer: Layer, B: int, R: int, T_cap: int) -> int:
    return _lib().kvc_workspace_bytes(layer.handle, B, R, T_cap)


def alloc_capsules(layer: Layer, B: int, R: int, device="cuda") -> torch.Tensor:
    return torch.empty(max(kvc_capsule_bytes(layer, B, R), 1), dtype=torch.uint8, device=device)


def alloc_workspace(layer: Layer, B: int, R: int, T_cap: int, device="cuda") -> torch.Tensor:
    return torch.empty(kvc_workspace_bytes(layer, B, R, T_cap), dtype=torch.uint8, device=device)


def kvc_layer_capsules_written(layer: Layer) -> None:
    """Call after anything but kvc_compress* has written into a capsule store used with this layer (see kvc.h)."""
    _check(_lib().kvc_layer_capsules_written(layer.handle), "kvc_layer_capsules_written")


def kvc_compress(layer: Layer, K_vis, V_vis, B: int, R: int, capsules, stream=None) -> None:
    _check(_lib().kvc_compress(layer.handle, _ptr(K_vis), _ptr(V_vis), B, R, _ptr(capsules), _stream(stream)),
           "kvc_compress")


def kvc_decode_attend(layer: Layer, q, capsules, B: int, R: int, K_txt, V_txt, T: int, T_cap: int, out,
                      workspace, stream=None) -> None:
    _check(_lib().kvc_decode_attend(layer.handle, _ptr(q), _ptr(capsules), B, R, _ptr(K_txt), _ptr(V_txt), T,
                                    T_cap, _ptr(out), _ptr(workspace), _stream(stream)), "kvc_decode_attend")


def kvc_compress_ragged(layer: Layer, K_vis, V_vis, B: int, N_cap: int, N_v, R_max: int, capsules, K_tail, V_tail,
                        T_cap: int, R_b, T_b, stream=None) -> None:
    """N_v, R_b, T_b: int32 device tensors of B entries (R_b and T_b are written)."""
    _check(_lib().kvc_compress_ragged(layer.handle, _ptr(K_vis), _ptr(V_vis), B, N_cap, _ptr(N_v), R_max, _ptr(capsules),
                                      _ptr(K_tail), _ptr(V_tail), T_cap, _ptr(R_b), _ptr(T_b), _stream(stream)),
           "kvc_compress_ragged")


def kvc_decode_attend_ragged(layer: Layer, q, capsules, B: int, R_max: int, R_b, K_txt, V_txt, T_max: int, T_b,
                             T_cap: int, out, workspace, stream=None) -> None:
    _check(_lib().kvc_decode_attend_ragged(layer.handle, _ptr(q), _ptr(capsules), B, R_max, _ptr(R_b), _ptr(K_txt),
                                           _ptr(V_txt), T_max, _ptr(T_b), T_cap, _ptr(out), _ptr(workspace),
                                           _stream(stream)), "kvc_decode_attend_ragged")


def kvc_decode_attend_static(layer: Layer, q, capsules, B: int, R: int, K_txt, V_txt, T: int, T_cap: int, out,
                             stream=None) -> None:
    """kvc_decode_attend for callers that cannot allocate a workspace: the scratch is a fixed array inside the
    library (kvc_static_scratch_bytes() bytes); larger shapes raise KvcError(-5).  Calls on one device share
    that array, so keep them stream-ordered."""
    _check(_lib().kvc_decode_attend_static(layer.handle, _ptr(q), _ptr(capsules), B, R, _ptr(K_txt), _ptr(V_txt),
                                           T, T_cap, _ptr(out), _stream(stream)), "kvc_decode_attend_static")


def kvc_static_scratch_bytes() -> int:
    return _lib().kvc_static_scratch_bytes()


def kvc_attend_full(layer: Layer, q, K, V, B: int, S: int, S_cap: int, out, workspace, stream=None) -> None:
    _check(_lib().kvc_attend_full(layer.handle, _ptr(q), _ptr(K), _ptr(V), B, S, S_cap, _ptr(out),
                                  _ptr(workspace), _stream(stream)), "kvc_attend_full")


def kvc_read_device_status(layer: Layer, B: int, R: int, T: int, workspace) -> int:
    out = C.c_int(-99)
    _check(_lib().kvc_read_device_status(layer.handle, B, R, T, _ptr(workspace), C.byref(out)),
           "kvc_read_device_status")
    return out.value


def kvc_read_compress_status(layer: Layer) -> int:
    out = C.c_int(-99)
    _check(_lib().kvc_read_compress_status(layer.handle, C.byref(out)), "kvc_read_compress_status")
    return out.value


def kvc_fit_value_pca(V_vis: torch.Tensor, n: int, m: int, want_eig: bool = False, stream=None):
    """FitValuePCA on the device.  V_vis [B, H_kv, R*n, d] -> (U [H_kv, m, n], mu [H_kv, d], eig [H_kv, n] fp64 or None,
    sweeps of the eigen-solver)."""
    B, H_kv, N_v, d = V_vis.shape
    if N_v % n:
        raise ValueError("N_v must be a whole number of n-token blocks")
    dev, dt = V_vis.device, V_vis.dtype
    U = torch.empty((H_kv, m, n), dtype=dt, device=dev)
    mu = torch.empty((H_kv, d), dtype=dt, device=dev)
    eig = torch.empty((H_kv, n), dtype=torch.float64, device=dev) if want_eig else None
    ws = torch.empty(_lib().kvc_fit_workspace_bytes(H_kv, n), dtype=torch.uint8, device=dev)
    sweeps = C.c_int(-1)
    _check(_lib().kvc_fit_value_pca(_ptr(V_vis.contiguous()), B, N_v // n, H_kv, n, m, _DTYPES[dt], _ptr(U), _ptr(mu), _ptr(eig),
                                    _ptr(ws), _stream(stream), C.byref(sweeps)), "kvc_fit_value_pca")
    return U, mu, eig, sweeps.value


def kvc_fit_key_reconstructor(K_vis: torch.Tensor, idx: torch.Tensor, n: int, rcond: float = 1e-10, stream=None):
    """Least-squares key reconstructor for the retained index set idx ([m] or [H_kv, m], host).  -> (theta [H_kv, m, n],
    sweeps of the eigen-solver)."""
    B, H_kv, N_v, d = K_vis.shape
    if N_v % n:
        raise ValueError("N_v must be a whole number of n-token blocks")
    dev, dt = K_vis.device, K_vis.dtype
    idx_host = idx.detach().to("cpu", torch.int32).contiguous()
    m = idx_host.shape[-1]
    theta = torch.empty((H_kv, m, n), dtype=dt, device=dev)
    ws = torch.empty(_lib().kvc_fit_workspace_bytes(H_kv, n), dtype=torch.uint8, device=dev)
    sweeps = C.c_int(-1)
    _check(_lib().kvc_fit_key_reconstructor(_ptr(K_vis.contiguous()), B, N_v // n, H_kv, n, m,
                                            C.cast(idx_host.data_ptr(), C.POINTER(C.c_int32)), 1 if idx_host.dim() == 2 else 0,
                                            float(rcond), _DTYPES[dt], _ptr(theta), _ptr(ws), _stream(stream), C.byref(sweeps)),
           "kvc_fit_key_reconstructor")
    return theta, sweeps.value


def kvc_collapse_theta(W1: torch.Tensor, W2: torch.Tensor, stream=None) -> torch.Tensor:
    """theta [H_kv, m, n] = W1 [H_kv, m, k] @ W2 [H_kv, k, n] on the device (a factored key reconstructor collapsed once,
    before kvc_layer_create)."""
    assert W1.is_cuda and W2.is_cuda and W1.dtype == W2.dtype and W1.is_contiguous() and W2.is_contiguous()
    H, m, k = W1.shape
    assert W2.shape[0] == H and W2.shape[1] == k
    n = W2.shape[2]
    theta = torch.empty((H, m, n), dtype=W1.dtype, device=W1.device)
    _check(_lib().kvc_collapse_theta(W1.data_ptr(), W2.data_ptr(), H, m, k, n, _DTYPES[W1.dtype], theta.data_ptr(), _stream(stream)),
           "kvc_collapse_theta")
    return theta


def kvc_selftest_bounded_wait(stream=None) -> int:
    """Status of a device-side wait that nothing completes: KVC_ERR_TIMEOUT (-7) when the bound works."""
    return int(_lib().kvc_selftest_bounded_wait(_stream(stream)))


def kvc_export_maps(layer: Layer, R: int):
    """(idx [H_kv, m] int32, group [R*n, 2] int32) as the device path holds them."""
    idx = torch.empty((layer.H_kv, layer.m), dtype=torch.int32)
    grp = torch.empty((R * layer.n, 2), dtype=torch.int32)
    _check(_lib().kvc_export_maps(layer.handle, R, C.cast(idx.data_ptr(), C.POINTER(C.c_int32)),
                                  C.cast(grp.data_ptr(), C.POINTER(C.c_int32))), "kvc_export_maps")
    return idx, grp


def capsule_views(layer: Layer, capsules, B: int, R: int):
    """(K_tilde [B,H_kv,R,m_k,d], V_tilde [B,H_kv,R,m_v,d]) typed views of a capsule store (no copy)."""
    total = kvc_capsule_bytes(layer, B, R)
    kb = total // (layer.m_k + layer.m_v) * layer.m_k
    return (capsules[:kb].view(layer.dtype).view(B, layer.H_kv, R, layer.m_k, layer.d),
            capsules[kb:total].view(layer.dtype).view(B, layer.H_kv, R, layer.m_v, layer.d))


KVC_KERNEL_COUNT = 14


def kvc_profile_start(max_launches: int) -> None:
    _check(_lib().kvc_profile_start(max_launches), "kvc_profile_start")


def kvc_profile_stop() -> None:
    _check(_lib().kvc_profile_stop(), "kvc_profile_stop")


def kvc_profile_read() -> dict:
    """{kernel name: (total_ms, launches)} of the bracketed launches; synchronise the stream first."""
    out = {}
    for k in range(KVC_KERNEL_COUNT):
        ms, n = C.c_double(), C.c_longlong()
        _check(_lib().kvc_profile_read(k, C.byref(ms), C.byref(n)), "kvc_profile_read")
        out[_lib().kvc_kernel_name(k).decode()] = (ms.value, n.value)
    return out
