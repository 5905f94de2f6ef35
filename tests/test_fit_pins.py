"""Pins of the fit oracle (oracle/kvcapsule_fit_oracle.py) against what the mathematics fixes.

FitValuePCA (Sec. 3.1 values paragraph, App. C Alg. 2) and the least-squares key reconstructor for a fixed index set
(the MSE term of Alg. 2).  A transposed operand, centring over the wrong axis, eigenvalues in the wrong order or a
missing block in the pooling fails at least one of these.
"""
import numpy as np
import pytest

from oracle import kvcapsule_fit_oracle as fit
from oracle import kvcapsule_oracle as orc


def _data(seed, B=3, H=2, R=2, n=10, d=6):
    r = np.random.default_rng(seed)
    return r, r.normal(size=(B, H, R * n, d)) * r.uniform(0.2, 3.0, size=(1, 1, R * n, 1))


def test_pca_is_eckart_young_optimal_and_residual_is_the_tail_of_the_spectrum():
    r, V = _data(1)
    n, m = 10, 4
    V += 5.0                                       # a mean that must be removed
    U, mu, eig = fit.fit_value_pca(V, n, m)
    for h in range(2):
        np.testing.assert_allclose(mu[h], V[:, h].reshape(-1, 6).mean(axis=0), atol=1e-13)
        np.testing.assert_allclose(U[h] @ U[h].T, np.eye(m), atol=1e-12)                 # orthonormal rows
        assert (np.diff(eig[h]) <= 1e-9).all()
    res = fit.value_residual_energy(V, U, mu, n)
    np.testing.assert_allclose(res, eig[:, m:].sum(axis=1), rtol=1e-10)
    # the residual written out block by block with the decode-side formulas: V_hat = U^T (U (V - mu)) + mu
    K_t, V_t = orc.compress(V, V, np.arange(m), U, mu, n)
    _, V_hat = orc.reconstruct(K_t, V_t, np.zeros((2, m, n)), U, mu)
    np.testing.assert_allclose(((V - V_hat) ** 2).sum(axis=(0, 2, 3)), res, rtol=1e-10)
    # no other rank-m orthonormal basis does better, and dropping the centring does worse or equal
    for _ in range(20):
        Q = np.linalg.qr(r.normal(size=(n, m)))[0].T
        other = fit.value_residual_energy(V, np.stack([Q, Q]), mu, n)
        assert (other >= res * (1 - 1e-12)).all()
    # total energy = sum of the spectrum
    Xc = V - mu[None, :, None, :]
    np.testing.assert_allclose((Xc ** 2).sum(axis=(0, 2, 3)), eig.sum(axis=1), rtol=1e-10)


def test_pca_recovers_a_planted_subspace_along_the_token_axis():
    """Blocks whose columns live in a known m-dimensional subspace of R^n that contains the all-ones direction (so the
    centring stays inside it): U spans exactly that subspace and the residual is zero.  The same data with the
    roles of the token and channel axes swapped in the fit would need rank min(n, d) instead."""
    r = np.random.default_rng(2)
    B, H, R, n, d, m = 4, 1, 3, 12, 5, 3
    raw = r.normal(size=(n, m))
    raw[:, 0] = 1.0
    basis = np.linalg.qr(raw)[0]                                        # n x m, orthonormal, spans the ones vector
    V = np.zeros((B, H, R * n, d))
    for b in range(B):
        for k in range(R):
            V[b, 0, k * n:(k + 1) * n] = basis @ r.normal(size=(m, d)) + r.normal(size=d)   # + a constant row
    U, mu, eig = fit.fit_value_pca(V, n, m)
    assert eig[0, m:].max() <= 1e-24 * eig[0, 0]
    np.testing.assert_allclose(U[0].T @ U[0], basis @ basis.T, atol=1e-10)
    assert fit.value_residual_energy(V, U, mu, n)[0] <= 1e-24 * eig[0].sum()
    assert fit.fit_value_pca(V, n, m - 1)[2][0, m - 1] > 1e-3 * eig[0, 0]   # one component fewer loses real energy


def test_pca_pools_every_block_of_every_sequence_and_ignores_their_order():
    r, V = _data(3, B=2, R=3)
    n, m = 10, 5
    U, mu, eig = fit.fit_value_pca(V, n, m)
    # the same blocks as six sequences of one block, in another order
    blocks = V.transpose(1, 0, 2, 3).reshape(2, 6, n, 6)[:, r.permutation(6)]
    V2 = blocks.transpose(1, 0, 2, 3)
    U2, mu2, eig2 = fit.fit_value_pca(V2, n, m)
    np.testing.assert_allclose(mu2, mu, atol=1e-13)
    np.testing.assert_allclose(eig2, eig, rtol=1e-10)
    for h in range(2):
        np.testing.assert_allclose(U2[h].T @ U2[h], U[h].T @ U[h], atol=1e-9)            # same projector


def test_least_squares_reconstructor_is_the_minimiser():
    r, K = _data(4, B=3, H=2, R=2, n=10, d=6)
    n, m = 10, 4
    idx = np.array([0, 3, 6, 9])
    theta = fit.fit_key_reconstructor(K, idx, n)
    base = fit.key_residual_energy(K, idx, theta, n)
    for h in range(2):
        X = fit.pooled_columns(K, n, h)
        grad = X[idx] @ (theta[h].T @ X[idx] - X).T                                       # d/dtheta of the loss / 2
        assert np.abs(grad).max() <= 1e-9 * np.abs(X).max() ** 2 * X.shape[1]
        np.testing.assert_allclose(theta[h][:, idx], np.eye(m), atol=1e-9)              # retained rows reproduce themselves
    for _ in range(10):
        worse = fit.key_residual_energy(K, idx, theta + 1e-3 * r.normal(size=theta.shape), n)
        assert (worse > base).all()
    # block by block with the decode-side formula K_hat = theta^T K_tilde
    K_t, V_t = orc.compress(K, K, idx, np.zeros((2, m, n)), np.zeros((2, 6)), n)
    K_hat, _ = orc.reconstruct(K_t, V_t, theta, np.zeros((2, m, n)), np.zeros((2, 6)))
    np.testing.assert_allclose(((K - K_hat) ** 2).sum(axis=(0, 2, 3)), base, rtol=1e-10)
    # per-head index sets
    idx2 = np.array([[0, 3, 6, 9], [1, 2, 5, 8]])
    th2 = fit.fit_key_reconstructor(K, idx2, n)
    np.testing.assert_allclose(th2[0], theta[0], atol=1e-12)
    np.testing.assert_allclose(th2[1][:, idx2[1]], np.eye(m), atol=1e-9)


def test_least_squares_recovers_an_exact_linear_dependence_and_handles_rank_deficiency():
    r = np.random.default_rng(5)
    B, R, n, d, m = 3, 2, 9, 7, 3
    idx = np.array([1, 4, 7])
    mix = r.normal(size=(n, m))
    mix[idx] = np.eye(m)
    K = np.zeros((B, 1, R * n, d))
    for b in range(B):
        for k in range(R):
            K[b, 0, k * n:(k + 1) * n] = mix @ r.normal(size=(m, d))
    theta = fit.fit_key_reconstructor(K, idx, n)
    np.testing.assert_allclose(theta[0], mix.T, atol=1e-9)
    assert fit.key_residual_energy(K, idx, theta, n)[0] <= 1e-20 * (K ** 2).sum()
    # two identical retained rows: the second-moment matrix is singular, the minimum-norm solution splits the weight
    K[:, :, 4::n] = K[:, :, 1::n]
    th = fit.fit_key_reconstructor(K, idx, n)
    assert np.isfinite(th).all()
    np.testing.assert_allclose(th[0][0], th[0][1], atol=1e-9)
    X = fit.pooled_columns(K, n, 0)
    np.testing.assert_allclose(th[0], np.linalg.pinv(X[idx].T) @ X.T, atol=1e-9)
