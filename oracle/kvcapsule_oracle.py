"""KVCapsule CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT PATH.

A plain, slow, fp64 numpy statement of what the KVCapsule decode-time hot path
computes, written from the paper (arxiv 2605.16439).  Only tests, the smoke
check and the benchmark's CPU-baseline leg may import it.  It shares no code
with the CUDA library and imports nothing from it.

Two forms of the decode step are given:

* Form 1 (`decode_attend_definition`) is the definition: reconstruct full-length
  vision keys and values from the capsules (Sec. 3.1 "Selective Retention and
  Reconstruction for Keys", "Sequence-Level Low-Rank Compression for Values"),
  concatenate with the untouched text K/V (Sec. 3.2 "Decoding Stage") and run
  the standard attention of Sec. 3.1's first equation.
* Form 2 (`decode_attend_fused`) takes Algorithm 1's steps in the paper's order
  and notation (scores in compressed space, expansion by theta, softmax,
  re-projection by U^T, product with the compressed values plus the mu term).

Readings of the paper taken here (each also listed in the design document):
  - f_theta acts linearly along the token axis: K_hat = theta^T K_tilde with one
    dense m x n matrix per KV head (Alg. 1 "MatMul(S_full, theta)" and App. D's
    theta in R^{H_kv x m x n} are only consistent with that).
  - the softmax runs jointly over all R*n reconstructed vision positions and
    the T text positions of a query head (Sec. 3.2 "Decoding Stage").
  - "rank R" of Alg. 1 = number of n-token vision blocks per sequence; theta, U,
    mu and the retained index set are shared by all blocks and sequences.
  - mu is a fixed per-(layer, KV head) vector (Sec. 3.2 first paragraph).
  - "P mu" in Alg. 1 step 4 = (sum_i P_i) mu^T.
  - compression ratio rho = 1 - l_r;  m = ceil(l_r n) in integer arithmetic on
    rho expressed in permille.
  - rho = 0 is a pass-through: capsules hold K and V verbatim.
  - the one-sided variants of App. G (Table 6) compress one side and keep the other verbatim:
    mode "k" stores the retained key rows and the full values (theta only), mode "v" the full keys
    and the projected values (U, mu only); mode "kv" is the method itself.
  - batches with per-sequence lengths (App. D: c, n, t are per-request quantities): sequence b has
    N_v[b] vision tokens and T[b] text tokens.  Compression works on whole n-token blocks (Sec. 3.1
    "an image with size n"); the paper does not say what happens to a vision run that is not a whole
    number of blocks.  Reading: the first floor(N_v[b] / n) blocks are compressed, the remaining
    N_v[b] mod n tokens are kept uncompressed and attended like text rows (placed in front of them).
    A sequence with no token at all gets a zero output row.

Parity pins: every function below is pinned by tests/test_oracle_pins.py
(library attention, lossless constructions, Eckart-Young, closed forms, brute
force, form 1 == form 2).  What is NOT pinned: behaviour with trained
parameters (no trained parameters exist here) -- "parity unpinned" for that.

Shapes (paper notation): q [B,H_q,d]; K_vis,V_vis [B,H_kv,R*n,d];
idx [m] or [H_kv,m]; theta,U [H_kv,m,n]; mu [H_kv,d];
K_tilde,V_tilde [B,H_kv,R,m,d]; K_txt,V_txt [B,H_kv,T,d]; out [B,H_q,d].
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# integer maps (Sec. 3.1: |M_l| = ceil(l_r n);  Alg. 1: Reshape to [B,H_kv,G,R,m])
# --------------------------------------------------------------------------
def retained_len(n: int, ratio_permille: int) -> int:
    """m = ceil(l_r * n) with l_r = 1 - rho, rho = ratio_permille / 1000, in integers."""
    if n <= 0 or not (0 <= ratio_permille < 1000):
        raise ValueError("need n > 0 and 0 <= ratio_permille < 1000")
    return (n * (1000 - ratio_permille) + 999) // 1000


def grouping_map(N_v: int, n: int) -> np.ndarray:
    """Vision token t (cache order) -> (block r, offset i): t = r*n + i.  int32 [N_v,2]."""
    if n <= 0 or N_v % n != 0:
        raise ValueError("N_v must be a whole number of n-token blocks")
    t = np.arange(N_v, dtype=np.int64)
    return np.stack([t // n, t % n], axis=1).astype(np.int32)


def _idx_for_head(idx: np.ndarray, h: int) -> np.ndarray:
    idx = np.asarray(idx)
    return idx[h] if idx.ndim == 2 else idx


# --------------------------------------------------------------------------
# standard attention (Sec. 3.1, first equation), single decode query, GQA
# --------------------------------------------------------------------------
def softmax(x: np.ndarray) -> np.ndarray:
    x = np.asarray(x, F64)
    e = np.exp(x - np.max(x))
    return e / np.sum(e)


def attention(q, K, V) -> np.ndarray:
    """softmax(q K^T / sqrt(d)) V per query head; query head hq reads KV head hq // G."""
    q, K, V = (np.asarray(a, F64) for a in (q, K, V))
    B, H_q, d = q.shape
    H_kv = K.shape[1]
    G = H_q // H_kv
    out = np.zeros((B, H_q, d), F64)
    for b in range(B):
        for hq in range(H_q):
            h = hq // G
            s = (K[b, h] @ q[b, hq]) / np.sqrt(F64(d))
            out[b, hq] = softmax(s) @ V[b, h]
    return out


# --------------------------------------------------------------------------
# prefill-stage compression (Sec. 3.2 "Prefilling Stage")
# --------------------------------------------------------------------------
def compress(K_vis, V_vis, idx, U, mu, n: int, passthrough: bool = False, mode: str = "kv"):
    """K_tilde = rows idx of each block's keys; V_tilde = U (V - 1 mu^T) per block.
    mode "k": only the keys are compressed (V_tilde = the block's values verbatim, n rows);
    mode "v": only the values (K_tilde = the block's keys verbatim, n rows)."""
    K_vis, V_vis = np.asarray(K_vis, F64), np.asarray(V_vis, F64)
    B, H_kv, N_v, d = K_vis.shape
    if N_v % n != 0:
        raise ValueError("N_v must be a whole number of n-token blocks")
    R = N_v // n
    if passthrough:
        return (K_vis.reshape(B, H_kv, R, n, d).copy(), V_vis.reshape(B, H_kv, R, n, d).copy())
    if mode != "k":
        U, mu = np.asarray(U, F64), np.asarray(mu, F64)
    m_k = n if mode == "v" else len(_idx_for_head(idx, 0))
    m_v = n if mode == "k" else U.shape[1]
    K_t = np.zeros((B, H_kv, R, m_k, d), F64)
    V_t = np.zeros((B, H_kv, R, m_v, d), F64)
    for b in range(B):
        for h in range(H_kv):
            for r in range(R):
                K_blk = K_vis[b, h, r * n:(r + 1) * n]
                V_blk = V_vis[b, h, r * n:(r + 1) * n]
                if mode == "v":
                    K_t[b, h, r] = K_blk
                else:
                    K_t[b, h, r] = K_blk[_idx_for_head(idx, h)]  # row selection by M_l
                if mode == "k":
                    V_t[b, h, r] = V_blk
                else:
                    V_center = V_blk - np.ones((n, 1), F64) * mu[h][None, :]
                    V_t[b, h, r] = U[h] @ V_center              # sequence-level PCA projection
    return K_t, V_t


# --------------------------------------------------------------------------
# decode-stage reconstruction (Sec. 3.2 "Decoding Stage")
# --------------------------------------------------------------------------
def reconstruct(K_t, V_t, theta, U, mu, passthrough: bool = False, mode: str = "kv"):
    """K_hat = theta^T K_tilde,  V_hat = U^T V_tilde + 1 mu^T;  returns [B,H_kv,R*n,d] each.
    The side a one-sided mode keeps verbatim is returned as stored."""
    K_t, V_t = np.asarray(K_t, F64), np.asarray(V_t, F64)
    B, H_kv, R, _, d = K_t.shape
    if passthrough:
        m = K_t.shape[3]
        return K_t.reshape(B, H_kv, R * m, d).copy(), V_t.reshape(B, H_kv, R * m, d).copy()
    n = K_t.shape[3] if mode == "v" else np.asarray(theta).shape[2]
    K_hat = np.zeros((B, H_kv, R * n, d), F64)
    V_hat = np.zeros((B, H_kv, R * n, d), F64)
    for b in range(B):
        for h in range(H_kv):
            for r in range(R):
                if mode == "v":
                    K_hat[b, h, r * n:(r + 1) * n] = K_t[b, h, r]
                else:
                    K_hat[b, h, r * n:(r + 1) * n] = np.asarray(theta[h], F64).T @ K_t[b, h, r]
                if mode == "k":
                    V_hat[b, h, r * n:(r + 1) * n] = V_t[b, h, r]
                else:
                    V_hat[b, h, r * n:(r + 1) * n] = (np.asarray(U[h], F64).T @ V_t[b, h, r]
                                                      + np.ones((n, 1), F64) * np.asarray(mu[h], F64)[None, :])
    return K_hat, V_hat


def collapse_reconstructor(W1, W2) -> np.ndarray:
    """A key reconstructor of two layers that are linear along the token axis (Sec. 3.1 calls f_theta a two-layer
    network; Alg. 1 step 2 and App. D use one m x n matrix theta per KV head):
        K_hat = W2^T (W1^T K_tilde) = (W1 W2)^T K_tilde,  so  theta[h] = W1[h] W2[h].
    W1 [H_kv, m, k], W2 [H_kv, k, n] -> theta [H_kv, m, n], the definition of the matrix product written out."""
    W1, W2 = np.asarray(W1, F64), np.asarray(W2, F64)
    H_kv, m, k = W1.shape
    n = W2.shape[2]
    theta = np.zeros((H_kv, m, n), F64)
    for h in range(H_kv):
        for j in range(m):
            for l in range(k):
                theta[h, j] += W1[h, j, l] * W2[h, l]
    return theta


def decode_attend_definition(q, K_t, V_t, theta, U, mu, K_txt, V_txt, passthrough: bool = False, mode: str = "kv"):
    """Form 1: reconstruct, concatenate with text K/V, run the original attention."""
    K_hat, V_hat = reconstruct(K_t, V_t, theta, U, mu, passthrough, mode)
    K_all = np.concatenate([K_hat, np.asarray(K_txt, F64)], axis=2)
    V_all = np.concatenate([V_hat, np.asarray(V_txt, F64)], axis=2)
    return attention(q, K_all, V_all)


# --------------------------------------------------------------------------
# Algorithm 1 (fused KVCapsule), with the text tail in the same softmax
# --------------------------------------------------------------------------
def decode_attend_fused(q, K_t, V_t, theta, U, mu, K_txt, V_txt, passthrough: bool = False, mode: str = "kv"):
    """Form 2: the associative order of Alg. 1 (steps 1-4) for one decode query per sequence.
    In a one-sided mode the side kept verbatim skips its step: mode "k" has no re-projection (the
    probabilities meet the n stored value rows directly), mode "v" no score expansion (the query meets
    all n stored keys).

    Nothing of length n x d is formed.  Per (sequence b, KV head h) and for the G query heads that read h:
      step 1  the query meets the m retained keys of every block:           s_c[g, r, j]
      step 2  those m scores are spread over the block's n positions by theta[h], and all R*n vision
              logits take part in ONE softmax together with the T text logits (Sec. 3.2, decoding stage)
      step 3  the vision probabilities are folded back to m weights per block by U[h]:  w_c[g, r, j]
      step 4  the weights meet the compressed values; the centring vector returns with the total vision
              probability as its coefficient; the text rows add their ordinary attention term.
    """
    q, K_t, V_t = np.asarray(q, F64), np.asarray(K_t, F64), np.asarray(V_t, F64)
    K_txt, V_txt = np.asarray(K_txt, F64), np.asarray(V_txt, F64)
    B, H_q, d = q.shape
    H_kv, R, m = K_t.shape[1], K_t.shape[2], K_t.shape[3]
    G = H_q // H_kv
    if passthrough:                      # rho = 0: theta = U = I, mu = 0
        theta = U = np.broadcast_to(np.eye(m, dtype=F64), (H_kv, m, m))
        mu = np.zeros((H_kv, d), F64)
    else:
        if mode == "v":                  # keys verbatim: the expansion is the identity on the n stored keys
            theta = np.broadcast_to(np.eye(m, dtype=F64), (H_kv, m, m))
        else:
            theta = np.asarray(theta, F64)
        if mode == "k":                  # values verbatim: no re-projection, no centring term
            nv = V_t.shape[3]
            U = np.broadcast_to(np.eye(nv, dtype=F64), (H_kv, nv, nv))
            mu = np.zeros((H_kv, d), F64)
        else:
            U, mu = np.asarray(U, F64), np.asarray(mu, F64)
    n = theta.shape[2]
    scale = 1.0 / np.sqrt(F64(d))
    out = np.zeros((B, H_q, d), F64)
    for b in range(B):
        for h in range(H_kv):
            for g in range(G):
                hq = h * G + g
                query = q[b, hq]
                # step 1
                s_c = np.zeros((R, m), F64)
                for r in range(R):
                    s_c[r] = (K_t[b, h, r] @ query) * scale
                # step 2
                logit_v = np.zeros((R, n), F64)
                for r in range(R):
                    logit_v[r] = s_c[r] @ theta[h]
                logit_t = (K_txt[b, h] @ query) * scale
                prob = softmax(np.concatenate([logit_v.reshape(R * n), logit_t]))
                prob_v, prob_t = prob[:R * n].reshape(R, n), prob[R * n:]
                # step 3
                w_c = np.zeros((R, U.shape[1]), F64)
                for r in range(R):
                    w_c[r] = U[h] @ prob_v[r]
                # step 4
                y = prob_v.sum() * mu[h]
                for r in range(R):
                    y = y + w_c[r] @ V_t[b, h, r]
                out[b, hq] = y + prob_t @ V_txt[b, h]
    return out


# --------------------------------------------------------------------------
# batches with per-sequence lengths
# --------------------------------------------------------------------------
def compress_ragged(K_vis, V_vis, N_v, idx, U, mu, n: int, R_max: int, mode: str = "kv"):
    """K_vis, V_vis [B,H_kv,N_cap,d] of which sequence b uses its first N_v[b] rows.
    Returns (K_tilde, V_tilde [B,H_kv,R_max,.,d] with zeros in the unused blocks, R_b [B] = whole blocks per
    sequence, K_tail, V_tail = lists of [H_kv, N_v[b] mod n, d] arrays: the rows left uncompressed)."""
    K_vis, V_vis = np.asarray(K_vis, F64), np.asarray(V_vis, F64)
    B = K_vis.shape[0]
    R_b = np.zeros(B, np.int64)
    K_t = V_t = None
    K_tail, V_tail = [], []
    for b in range(B):
        R_b[b] = int(N_v[b]) // n
        if R_b[b] > R_max:
            raise ValueError("R_max is smaller than a sequence's block count")
        whole = int(R_b[b]) * n
        # the sequence's whole blocks, compressed as a batch of one
        Kb, Vb = compress(K_vis[b:b + 1, :, :whole], V_vis[b:b + 1, :, :whole], idx, U, mu, n, False, mode)
        if K_t is None:
            K_t = np.zeros((B, Kb.shape[1], R_max, Kb.shape[3], Kb.shape[4]), F64)
            V_t = np.zeros((B, Vb.shape[1], R_max, Vb.shape[3], Vb.shape[4]), F64)
        K_t[b, :, :R_b[b]] = Kb[0]
        V_t[b, :, :R_b[b]] = Vb[0]
        K_tail.append(K_vis[b, :, whole:int(N_v[b])].copy())
        V_tail.append(V_vis[b, :, whole:int(N_v[b])].copy())
    return K_t, V_t, R_b, K_tail, V_tail


def decode_attend_ragged(q, K_t, V_t, theta, U, mu, K_txt, V_txt, R_b, T_b, mode: str = "kv"):
    """Decode step on a padded batch: sequence b attends to its first R_b[b] blocks of the capsule store
    [B,H_kv,R_max,.,d] and to the first T_b[b] rows of K_txt, V_txt [B,H_kv,T_cap,d].  Written as ONE masked
    softmax over the padded axis (positions a sequence does not have get probability exactly zero); the pin is that
    this equals running every sequence alone with its own lengths."""
    q = np.asarray(q, F64)
    K_txt, V_txt = np.asarray(K_txt, F64), np.asarray(V_txt, F64)
    K_hat, V_hat = reconstruct(K_t, V_t, theta, U, mu, False, mode)        # [B,H_kv,R_max*n,d]
    B, H_q, d = q.shape
    H_kv = K_hat.shape[1]
    G = H_q // H_kv
    n = K_hat.shape[2] // np.asarray(K_t).shape[2] if np.asarray(K_t).shape[2] else 0
    out = np.zeros((B, H_q, d), F64)
    for b in range(B):
        have_v = np.arange(K_hat.shape[2]) < int(R_b[b]) * n
        have_t = np.arange(K_txt.shape[2]) < int(T_b[b])
        have = np.concatenate([have_v, have_t])
        if not have.any():
            continue
        for hq in range(H_q):
            h = hq // G
            K_all = np.concatenate([K_hat[b, h], K_txt[b, h]], axis=0)
            V_all = np.where(have[:, None], np.concatenate([V_hat[b, h], V_txt[b, h]], axis=0), 0.0)
            logit = np.where(have, (K_all @ q[b, hq]) / np.sqrt(d), -np.inf)
            prob = np.where(have, np.exp(logit - logit[have].max()), 0.0)
            out[b, hq] = (prob / prob.sum()) @ V_all
    return out


# --------------------------------------------------------------------------
# persistent-memory footprint of one layer (App. D, Eqs. 1-2)
# --------------------------------------------------------------------------
def footprint_base(B, H_kv, c, n_vis, t, d, b_kv) -> int:
    """Eq. 1: 2 B H_kv (c + n + t) d b_kv."""
    return 2 * B * H_kv * (c + n_vis + t) * d * b_kv


def footprint_kvcapsule(B, H_kv, c, n, R, t, d, b_kv, ratio_permille, b_param=None) -> int:
    """Eq. 2 with R blocks of n tokens: compressed cache + S_recon(theta) + S_PCA(U, mu)."""
    b_param = b_kv if b_param is None else b_param
    m = retained_len(n, ratio_permille)
    cache = 2 * B * H_kv * (c + R * m + t) * d * b_kv
    s_recon = H_kv * m * n * b_param
    s_pca = H_kv * m * n * b_param + H_kv * d * b_param
    return cache + s_recon + s_pca
