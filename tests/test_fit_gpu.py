"""The device fits (FitValuePCA, least-squares key reconstructor) against the fit oracle, through the C ABI.

What is unique is compared: the mean, the spectrum, the projector onto the kept subspace, the energy the fitted
parameters lose (evaluated by the oracle in fp64 from the device's outputs).  Eigenvector signs are a convention, checked
on its own.
"""
import numpy as np
import pytest
import torch

from oracle import kvcapsule_fit_oracle as fit
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


SHAPES = [  # B, H_kv, R, grid, m
    (3, 2, 2, 6, 15),
    (2, 3, 3, 5, 10),        # n = 25: odd, the solver pads one index
    (4, 2, 2, 12, 58),       # n = 144
    (2, 1, 1, 4, 16),        # m = n
    (1, 2, 1, 3, 1),         # n = 9, m = 1: a single component
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,H,R,grid,m", SHAPES)
def test_value_pca_matches_the_svd(B, H, R, grid, m, dtype):
    n = grid * grid
    dt = wl.torch_dtype(dtype)
    V = wl.vision_kv(B, H, R, grid, 128, 77 + grid, "cpu", dt) + torch.tensor(0.75, dtype=dt)
    U_g, mu_g, eig_g, sweeps = kvc.kvc_fit_value_pca(V.to(DEV), n, m, want_eig=True)
    assert 0 < sweeps < 40
    V64 = tl.np64(V)
    U_o, mu_o, eig_o = fit.fit_value_pca(V64, n, m)
    half_ulp = 2.0 ** -24 if dtype == "f32" else 2.0 ** -8        # of the magnitude: 24 / 8 significant bits
    np.testing.assert_allclose(tl.np64(mu_g), mu_o, atol=half_ulp * np.abs(mu_o).max() * 1.01 + 1e-12)
    eig = eig_g.cpu().numpy()
    np.testing.assert_allclose(eig, eig_o, atol=1e-9 * eig_o[:, :1].max(), rtol=1e-9)
    U = tl.np64(U_g)
    # sign convention: the entry of largest magnitude of every row is positive
    big = np.take_along_axis(U, np.abs(U).argmax(axis=2)[..., None], axis=2)
    assert (big > 0).all()
    if dtype == "f32":
        for h in range(H):
            np.testing.assert_allclose(U[h] @ U[h].T, np.eye(m), atol=2e-6)
        # the energy the device's (U, mu) lose, against the tail of the oracle's spectrum
        res = fit.value_residual_energy(V64, U, tl.np64(mu_g), n)
        want = eig_o[:, m:].sum(axis=1)
        np.testing.assert_allclose(res, want, rtol=1e-3, atol=1e-9 * eig_o.sum(axis=1).max())
        if m < n:
            gap = (eig_o[:, m - 1] - eig_o[:, m]) / eig_o[:, 0]
            for h in range(H):
                if gap[h] > 1e-3:
                    np.testing.assert_allclose(U[h].T @ U[h], U_o[h].T @ U_o[h], atol=1e-5 / gap[h])
    else:
        # bf16 storage rounds every entry: the projector moves by about 2^-8 of its entries' scale
        res = fit.value_residual_energy(V64, U, tl.np64(mu_g), n)
        total = eig_o.sum(axis=1)
        want = eig_o[:, m:].sum(axis=1)
        assert (np.abs(res - want) <= 2e-2 * total).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,H,R,grid,m", SHAPES[:4])
@pytest.mark.parametrize("per_head", [False, True])
def test_key_reconstructor_matches_least_squares(B, H, R, grid, m, dtype, per_head):
    n = grid * grid
    dt = wl.torch_dtype(dtype)
    K = wl.vision_kv(B, H, R, grid, 128, 99 + grid, "cpu", dt)
    idx = wl.random_sorted_idx(n, m, 5 + grid, H if per_head else 0)
    theta_g, sweeps = kvc.kvc_fit_key_reconstructor(K.to(DEV), idx, n)
    assert 0 < sweeps < 40
    K64 = tl.np64(K)
    theta_o = fit.fit_key_reconstructor(K64, idx.numpy(), n)
    th = tl.np64(theta_g)
    best = fit.key_residual_energy(K64, idx.numpy(), theta_o, n)
    got = fit.key_residual_energy(K64, idx.numpy(), th, n)
    total = (K64 ** 2).sum(axis=(0, 2, 3))
    if dtype == "f32":
        np.testing.assert_allclose(got, best, rtol=1e-3, atol=1e-10 * total.max())
        np.testing.assert_allclose(th, theta_o, atol=2e-5 * max(1.0, np.abs(theta_o).max()))
    else:
        np.testing.assert_allclose(th, theta_o, atol=2.0 ** -8 * max(1.0, np.abs(theta_o).max()))
        assert (got <= best + 1e-3 * total).all()
    assert (got >= best * (1 - 1e-9)).all()          # nothing beats the minimiser


def test_fitted_parameters_through_the_decode_path():
    """Fitted on one set of blocks, used on another: the ordinary parity check with the device-fitted parameters, and
    the compressed output close to full attention where the data is redundant (smoothed fields)."""
    shape = wl.Shape("fit", 1, 2, 4, 2, 128, 12, 3, 16, 1, "f32", 600)
    n, m = shape.n, orc.retained_len(shape.n, 600)
    train_K = wl.vision_kv(6, 2, 4, 12, 128, 501, DEV)
    train_V = wl.vision_kv(6, 2, 4, 12, 128, 502, DEV)
    idx = wl.evenly_spaced_idx(n, m)
    U, mu, _, _ = kvc.kvc_fit_value_pca(train_V, n, m)
    theta, _ = kvc.kvc_fit_key_reconstructor(train_K, idx, n)
    p = tl.make_problem(shape, 503)
    p.update(theta=theta.cpu(), U=U.cpu(), mu=mu.cpu(), idx=idx)
    K_o, V_o, out_o = tl.oracle_run(shape, p)
    layer, K_g, V_g, out_g = tl.gpu_run(shape, p)
    tl.assert_close(tl.np64(out_g), out_o, "f32", "decode with fitted parameters")
    K_all = np.concatenate([tl.np64(p["K_vis"]), tl.np64(p["K_txt"])], axis=2)
    V_all = np.concatenate([tl.np64(p["V_vis"]), tl.np64(p["V_txt"])], axis=2)
    full = orc.attention(tl.np64(p["q"]), K_all, V_all)
    cos = (full * out_o).sum(-1) / np.linalg.norm(full, axis=-1) / np.linalg.norm(out_o, axis=-1)
    rand = tl.oracle_run(shape, tl.make_problem(shape, 503))[2]
    cos_rand = (full * rand).sum(-1) / np.linalg.norm(full, axis=-1) / np.linalg.norm(rand, axis=-1)
    assert cos.min() > 0.9 and cos.mean() > cos_rand.mean() + 0.3


def test_fit_argument_errors():
    V = torch.zeros((1, 1, 16, 128), device=DEV)
    lib = kvc._lib()
    ws = torch.empty(lib.kvc_fit_workspace_bytes(1, 16), dtype=torch.uint8, device=DEV)
    U = torch.empty((1, 4, 16), device=DEV)
    mu = torch.empty((1, 128), device=DEV)
    call = lambda *a: lib.kvc_fit_value_pca(*a)
    assert call(None, 1, 1, 1, 16, 4, 0, U.data_ptr(), mu.data_ptr(), None, ws.data_ptr(), None, None) == -1
    assert call(V.data_ptr(), 1, 1, 1, 16, 17, 0, U.data_ptr(), mu.data_ptr(), None, ws.data_ptr(), None, None) == -2
    assert call(V.data_ptr(), 1, 1, 1, 16, 4, 5, U.data_ptr(), mu.data_ptr(), None, ws.data_ptr(), None, None) == -3
    assert call(V.data_ptr(), 1, 1, 1, 16, 4, 0, U.data_ptr(), mu.data_ptr(), None, ws.data_ptr() + 8, None, None) == -5
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_fit_key_reconstructor(V, torch.tensor([3, 2, 5]), 16)
    assert e.value.status == -8
    assert lib.kvc_fit_workspace_bytes(0, 16) == 0
