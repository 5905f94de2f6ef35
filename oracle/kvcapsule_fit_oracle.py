"""KVCapsule CPU oracle for the parameter fits -- TEST INFRASTRUCTURE, NOT THE PRODUCT PATH.

Plain fp64 numpy statements of the two fits that produce a layer's parameters from activations, written from the
paper (arxiv 2605.16439).  Only tests, the smoke check and the benchmark's CPU-baseline leg may import it.  It shares
no code with the CUDA library and imports nothing from it.

* `fit_value_pca`: FitValuePCA of App. C, Alg. 2, as Sec. 3.1 "Sequence-Level Low-Rank Compression for Values" states it:
  a mean vector mu over the sequence axis, then PCA along the sequence dimension of the centred values by singular
  value decomposition, keeping the top m components; U is m x n.
* `fit_key_reconstructor`: the key reconstructor for a FIXED retained index set as the minimiser of the reconstruction
  loss MSE(K_hat, K) of Alg. 2, K_hat = theta^T K[idx].

Readings of the paper taken here (each also listed in the design document):
  - the "dataset" of Alg. 2 is a set of n-token blocks; all blocks of all sequences are pooled per KV head.
  - mu is ONE vector per (layer, KV head) (Sec. 3.2: the centring vectors are fixed at inference): the mean over the
    pooled blocks and their n positions.
  - "PCA along the sequence dimension": the n token positions are the variables and every (block, channel) column of
    the centred n x d value matrices is an observation, so the principal directions are the left singular vectors of
    the n x (blocks d) matrix of pooled columns and U's rows are the top m of them.
  - the paper trains f_theta (a two-layer MLP, which acts linearly along the token axis here) and the mask jointly by
    gradient descent on MSE plus mask losses; with the mask fixed and a linear reconstructor the MSE term has a closed
    minimiser, the least-squares solution below (minimum-norm when the retained rows are rank deficient).  The mask
    search itself is not part of this oracle.

Parity pins (tests/test_fit_pins.py): Eckart-Young optimality and the residual identity sum_{i>m} s_i^2, recovery of a
planted subspace, invariance to the order of blocks, zero gradient of the loss and strict increase under perturbation,
exact recovery when every key row is a combination of retained rows, agreement with the explicit stacked design matrix.

Shapes: V_vis, K_vis [B, H_kv, R*n, d]; U, theta [H_kv, m, n]; mu [H_kv, d]; eig [H_kv, n].
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def pooled_columns(X_vis, n: int, h: int) -> np.ndarray:
    """The n x (B R d) matrix whose columns are the (block, channel) columns of KV head h."""
    X_vis = np.asarray(X_vis, F64)
    B, _, N_v, d = X_vis.shape
    R = N_v // n
    blocks = X_vis[:, h].reshape(B * R, n, d)              # every n-token block of every sequence
    return np.concatenate(list(blocks), axis=1)            # [n, B R d]


def fit_value_pca(V_vis, n: int, m: int):
    """(U [H_kv,m,n], mu [H_kv,d], eig [H_kv,n]): eig = squared singular values of the pooled centred columns,
    descending; the energy the rank-m projection loses is eig[m:].sum() (Eckart-Young)."""
    V_vis = np.asarray(V_vis, F64)
    _, H_kv, _, d = V_vis.shape
    U = np.zeros((H_kv, m, n), F64)
    mu = np.zeros((H_kv, d), F64)
    eig = np.zeros((H_kv, n), F64)
    for h in range(H_kv):
        mu[h] = V_vis[:, h].reshape(-1, d).mean(axis=0)
        X = pooled_columns(V_vis - mu[None, :, None, :], n, h)
        W, s, _ = np.linalg.svd(X, full_matrices=False)
        U[h] = W[:, :m].T
        eig[h, :len(s)] = s ** 2
    return U, mu, eig


def value_residual_energy(V_vis, U, mu, n: int) -> np.ndarray:
    """[H_kv]: sum over blocks of || X - U^T U X ||_F^2 for X = the centred block."""
    V_vis, U, mu = np.asarray(V_vis, F64), np.asarray(U, F64), np.asarray(mu, F64)
    out = np.zeros(U.shape[0], F64)
    for h in range(U.shape[0]):
        X = pooled_columns(V_vis - mu[None, :, None, :], n, h)
        out[h] = ((X - U[h].T @ (U[h] @ X)) ** 2).sum()
    return out


def fit_key_reconstructor(K_vis, idx, n: int, rcond: float = 1e-10):
    """theta [H_kv,m,n] minimising sum over blocks of || K - theta^T K[idx] ||_F^2 (minimum-norm solution; directions
    of the retained rows' second-moment matrix whose eigenvalue is below rcond times the largest are dropped)."""
    K_vis = np.asarray(K_vis, F64)
    H_kv = K_vis.shape[1]
    idx = np.asarray(idx)
    m = idx.shape[-1]
    theta = np.zeros((H_kv, m, n), F64)
    for h in range(H_kv):
        sel = idx[h] if idx.ndim == 2 else idx
        X = pooled_columns(K_vis, n, h)                    # [n, N]
        Xr = X[sel]                                        # retained rows [m, N]
        # each column is one observation: retained entries -> all n entries, K_col = theta^T Kr_col
        theta[h] = np.linalg.lstsq(Xr.T, X.T, rcond=np.sqrt(rcond))[0]
    return theta


def key_residual_energy(K_vis, idx, theta, n: int) -> np.ndarray:
    K_vis, theta = np.asarray(K_vis, F64), np.asarray(theta, F64)
    idx = np.asarray(idx)
    out = np.zeros(theta.shape[0], F64)
    for h in range(theta.shape[0]):
        sel = idx[h] if idx.ndim == 2 else idx
        X = pooled_columns(K_vis, n, h)
        out[h] = ((X - theta[h].T @ X[sel]) ** 2).sum()
    return out
