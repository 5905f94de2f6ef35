"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each pin is chosen so that a
plausible slip in the oracle (dropped mu term, wrong sign, wrong index set,
transposed operand, wrong GQA head map, missing 1/sqrt(d), separate instead of
joint softmax, wrong block order) fails at least one of them.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import kvcapsule_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _library_attention(q, K, V):
    """torch's fp64 scaled-dot-product attention as an independent library routine."""
    B, H_q, d = q.shape
    G = H_q // K.shape[1]
    qt = torch.from_numpy(np.ascontiguousarray(q)).reshape(B, H_q, 1, d)
    Kt = torch.from_numpy(np.ascontiguousarray(K)).repeat_interleave(G, dim=1)
    Vt = torch.from_numpy(np.ascontiguousarray(V)).repeat_interleave(G, dim=1)
    out = torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt)
    return out.reshape(B, H_q, d).numpy()


def _problem(seed, B=2, H_q=6, H_kv=2, d=8, n=12, m=5, R=3, T=4):
    r = _rng(seed)
    return dict(
        q=r.standard_normal((B, H_q, d)),
        K_vis=r.standard_normal((B, H_kv, R * n, d)),
        V_vis=r.standard_normal((B, H_kv, R * n, d)),
        K_txt=r.standard_normal((B, H_kv, T, d)),
        V_txt=r.standard_normal((B, H_kv, T, d)),
        theta=r.standard_normal((H_kv, m, n)) / math.sqrt(d),
        U=r.standard_normal((H_kv, m, n)) / math.sqrt(d),
        mu=r.standard_normal((H_kv, d)),
        idx=np.sort(r.permutation(n)[:m]).astype(np.int32),
        n=n, m=m, R=R, T=T,
    )


# ---------------------------------------------------------------- integer maps
def test_retained_len_table():
    # m = ceil((1 - rho) n), Sec. 3.1; the values used by every configuration
    assert orc.retained_len(576, 600) == 231
    assert orc.retained_len(1024, 600) == 410
    assert orc.retained_len(256, 600) == 103
    assert [orc.retained_len(1024, r) for r in (0, 200, 400, 600, 800)] == [1024, 820, 615, 410, 205]
    for n in (1, 7, 576, 1000, 1024):
        for r in (0, 1, 333, 500, 950, 999):
            m = orc.retained_len(n, r)
            assert m == math.ceil(n * (1000 - r) / 1000)          # exact rational ceil
            assert 1 <= m <= n
    with pytest.raises(ValueError):
        orc.retained_len(16, 1000)


def test_grouping_map_is_block_decomposition():
    g = orc.grouping_map(3 * 7, 7)
    assert g.dtype == np.int32 and g.shape == (21, 2)
    for t in range(21):
        assert g[t, 0] * 7 + g[t, 1] == t and 0 <= g[t, 1] < 7
    with pytest.raises(ValueError):
        orc.grouping_map(20, 7)


# ---------------------------------------------------------------- attention vs a library
@pytest.mark.parametrize("seed", [0, 1])
def test_attention_matches_library_routine(seed):
    r = _rng(seed)
    q = r.standard_normal((2, 6, 16))
    K = r.standard_normal((2, 3, 37, 16))
    V = r.standard_normal((2, 3, 37, 16))
    np.testing.assert_allclose(orc.attention(q, K, V), _library_attention(q, K, V), atol=1e-13)


def test_softmax_invariants():
    r = _rng(3)
    x = r.standard_normal(50) * 5
    p = orc.softmax(x)
    assert abs(p.sum() - 1.0) < 1e-12 and (p >= 0).all()
    np.testing.assert_allclose(orc.softmax(x + 123.456), p, atol=1e-13)
    # closed form on two logits: logistic function
    a, b = 0.3, -1.1
    np.testing.assert_allclose(orc.softmax(np.array([a, b]))[0], 1 / (1 + math.exp(b - a)), atol=1e-15)


def test_output_lies_in_value_hull():
    p = _problem(4)
    K_t, V_t = orc.compress(p["K_vis"], p["V_vis"], p["idx"], p["U"], p["mu"], p["n"])
    K_hat, V_hat = orc.reconstruct(K_t, V_t, p["theta"], p["U"], p["mu"])
    out = orc.decode_attend_definition(p["q"], K_t, V_t, p["theta"], p["U"], p["mu"], p["K_txt"], p["V_txt"])
    V_all = np.concatenate([V_hat, p["V_txt"]], axis=2)
    G = p["q"].shape[1] // V_all.shape[1]
    for hq in range(p["q"].shape[1]):
        lo, hi = V_all[:, hq // G].min(axis=1), V_all[:, hq // G].max(axis=1)
        assert (out[:, hq] >= lo - 1e-12).all() and (out[:, hq] <= hi + 1e-12).all()


# ---------------------------------------------------------------- limit cases of the whole path
def test_ratio_zero_is_uncompressed_attention_exactly():
    p = _problem(5)
    K_t, V_t = orc.compress(p["K_vis"], p["V_vis"], None, None, None, p["n"], passthrough=True)
    assert K_t.shape == (2, 2, p["R"], p["n"], 8)
    out = orc.decode_attend_definition(p["q"], K_t, V_t, None, None, None, p["K_txt"], p["V_txt"], passthrough=True)
    K_all = np.concatenate([p["K_vis"], p["K_txt"]], axis=2)
    V_all = np.concatenate([p["V_vis"], p["V_txt"]], axis=2)
    assert np.array_equal(out, orc.attention(p["q"], K_all, V_all))          # bit for bit
    np.testing.assert_allclose(out, _library_attention(p["q"], K_all, V_all), atol=1e-13)
    fused = orc.decode_attend_fused(p["q"], K_t, V_t, None, None, None, p["K_txt"], p["V_txt"], passthrough=True)
    np.testing.assert_allclose(fused, out, atol=1e-13)


def test_no_vision_blocks_is_text_attention():
    p = _problem(6, R=0)
    K_t = np.zeros((2, 2, 0, p["m"], 8))
    for f in (orc.decode_attend_definition, orc.decode_attend_fused):
        out = f(p["q"], K_t, K_t, p["theta"], p["U"], p["mu"], p["K_txt"], p["V_txt"])
        np.testing.assert_allclose(out, _library_attention(p["q"], p["K_txt"], p["V_txt"]), atol=1e-13)


# ---------------------------------------------------------------- lossless constructions
def _lossless_key_side(p, r):
    """theta with theta[:, idx] = I_m and K = theta^T C  =>  K_hat == K."""
    H_kv, m, n = p["theta"].shape
    theta = p["theta"].copy()
    for h in range(H_kv):
        theta[h][:, p["idx"]] = np.eye(m)
    B, _, N_v, d = p["K_vis"].shape
    C = r.standard_normal((B, H_kv, p["R"], m, d))
    K_vis = np.einsum("hmn,bhrmd->bhrnd", theta, C).reshape(B, H_kv, N_v, d)
    return theta, K_vis


def _lossless_value_side(p, r):
    """U with orthonormal rows and V = U^T C + 1 mu^T  =>  V_hat == V."""
    H_kv, m, n = p["U"].shape
    U = np.stack([np.linalg.qr(r.standard_normal((n, m)))[0].T for _ in range(H_kv)])
    B, _, N_v, d = p["V_vis"].shape
    C = r.standard_normal((B, H_kv, p["R"], m, d))
    V_vis = np.einsum("hmn,bhrmd->bhrnd", U, C) + p["mu"][None, :, None, None, :]
    return U, V_vis.reshape(B, H_kv, N_v, d)


def test_lossless_parameters_reproduce_full_attention():
    p = _problem(7)
    r = _rng(70)
    theta, K_vis = _lossless_key_side(p, r)
    U, V_vis = _lossless_value_side(p, r)
    K_t, V_t = orc.compress(K_vis, V_vis, p["idx"], U, p["mu"], p["n"])
    K_hat, V_hat = orc.reconstruct(K_t, V_t, theta, U, p["mu"])
    np.testing.assert_allclose(K_hat, K_vis, atol=1e-12)
    np.testing.assert_allclose(V_hat, V_vis, atol=1e-12)
    K_all = np.concatenate([K_vis, p["K_txt"]], axis=2)
    V_all = np.concatenate([V_vis, p["V_txt"]], axis=2)
    want = _library_attention(p["q"], K_all, V_all)
    for f in (orc.decode_attend_definition, orc.decode_attend_fused):
        got = f(p["q"], K_t, V_t, theta, U, p["mu"], p["K_txt"], p["V_txt"])
        np.testing.assert_allclose(got, want, atol=1e-11)


def test_per_head_index_sets():
    p = _problem(8)
    r = _rng(80)
    idx2 = np.stack([np.sort(r.permutation(p["n"])[:p["m"]]) for _ in range(2)]).astype(np.int32)
    assert not np.array_equal(idx2[0], idx2[1])
    K_t, _ = orc.compress(p["K_vis"], p["V_vis"], idx2, p["U"], p["mu"], p["n"])
    for h in range(2):
        for blk in range(p["R"]):
            for j in range(p["m"]):
                assert np.array_equal(K_t[1, h, blk, j], p["K_vis"][1, h, blk * p["n"] + idx2[h, j]])


def test_value_pca_is_eckart_young_optimal():
    # U = top-m left singular vectors of the centred block (Sec. 3.1): the residual
    # energy of the re-projection equals the discarded singular values' energy.
    r = _rng(9)
    n, m, d = 24, 7, 10
    V = r.standard_normal((1, 1, n, d)) @ np.diag(np.linspace(2, 0.1, d))
    mu = V.mean(axis=2)[0]                                  # [1,d]
    Uf, s, _ = np.linalg.svd(V[0, 0] - mu, full_matrices=False)
    U = Uf[:, :m].T[None]                                   # [1,m,n]
    _, V_t = orc.compress(V, V, np.arange(m), U, mu, n)
    _, V_hat = orc.reconstruct(V_t, V_t, U, U, mu)
    resid = np.sum((V - V_hat) ** 2)
    np.testing.assert_allclose(resid, np.sum(s[m:] ** 2), rtol=1e-10)


# ---------------------------------------------------------------- one-sided variants (App. G)
def test_one_sided_modes():
    """Mode "k" (keys compressed, values verbatim) and mode "v" (values compressed, keys verbatim): (i) each equals the
    two-sided method given the identity on the side it keeps (U = I_n, mu = 0, or theta = I_n with every index
    retained), which ties them to the pinned two-sided path; (ii) with the lossless construction on the compressed
    side they reproduce full attention through the library routine; (iii) definition == Alg. 1 order."""
    p = _problem(21)
    r = _rng(210)
    n, m, H_kv, d = p["n"], p["m"], 2, 8
    eye_n = np.broadcast_to(np.eye(n), (H_kv, n, n))
    K_all = lambda Kv: np.concatenate([Kv, p["K_txt"]], axis=2)
    V_all = lambda Vv: np.concatenate([Vv, p["V_txt"]], axis=2)
    # ---- mode "k"
    K_t, V_t = orc.compress(p["K_vis"], p["V_vis"], p["idx"], None, None, n, mode="k")
    assert K_t.shape[3] == m and V_t.shape[3] == n
    assert np.array_equal(V_t.reshape(p["V_vis"].shape), p["V_vis"])
    a = orc.decode_attend_definition(p["q"], K_t, V_t, p["theta"], None, None, p["K_txt"], p["V_txt"], mode="k")
    b = orc.decode_attend_fused(p["q"], K_t, V_t, p["theta"], None, None, p["K_txt"], p["V_txt"], mode="k")
    np.testing.assert_allclose(a, b, atol=1e-10)
    K2, V2 = orc.compress(p["K_vis"], p["V_vis"], p["idx"], eye_n, np.zeros((H_kv, d)), n)
    c = orc.decode_attend_definition(p["q"], K2, V2, p["theta"], eye_n, np.zeros((H_kv, d)), p["K_txt"], p["V_txt"])
    np.testing.assert_allclose(a, c, atol=1e-12)
    theta_l, K_l = _lossless_key_side(p, r)
    K_t, V_t = orc.compress(K_l, p["V_vis"], p["idx"], None, None, n, mode="k")
    got = orc.decode_attend_fused(p["q"], K_t, V_t, theta_l, None, None, p["K_txt"], p["V_txt"], mode="k")
    np.testing.assert_allclose(got, _library_attention(p["q"], K_all(K_l), V_all(p["V_vis"])), atol=1e-11)
    # ---- mode "v"
    K_t, V_t = orc.compress(p["K_vis"], p["V_vis"], None, p["U"], p["mu"], n, mode="v")
    assert K_t.shape[3] == n and V_t.shape[3] == m
    assert np.array_equal(K_t.reshape(p["K_vis"].shape), p["K_vis"])
    a = orc.decode_attend_definition(p["q"], K_t, V_t, None, p["U"], p["mu"], p["K_txt"], p["V_txt"], mode="v")
    b = orc.decode_attend_fused(p["q"], K_t, V_t, None, p["U"], p["mu"], p["K_txt"], p["V_txt"], mode="v")
    np.testing.assert_allclose(a, b, atol=1e-10)
    # the two-sided method with every key retained and theta = I_n, on the same U and mu
    K2 = p["K_vis"].reshape(2, H_kv, p["R"], n, d)
    c = orc.decode_attend_definition(p["q"], K2, V_t, eye_n, p["U"], p["mu"], p["K_txt"], p["V_txt"])
    np.testing.assert_allclose(a, c, atol=1e-12)
    U_l, V_l = _lossless_value_side(p, r)
    K_t, V_t = orc.compress(p["K_vis"], V_l, None, U_l, p["mu"], n, mode="v")
    got = orc.decode_attend_fused(p["q"], K_t, V_t, None, U_l, p["mu"], p["K_txt"], p["V_txt"], mode="v")
    np.testing.assert_allclose(got, _library_attention(p["q"], K_all(p["K_vis"]), V_all(V_l)), atol=1e-11)


# ---------------------------------------------------------------- per-sequence lengths
def test_ragged_batch_equals_the_sequences_run_one_by_one():
    """A padded batch with per-sequence block counts and text lengths (masked softmax) gives, for every sequence, what
    the uniform functions give for that sequence alone with its own R and T; padding contents (NaN here) never leak;
    the limits R = 0 (text only), T = 0 (vision only) and an empty sequence (zero row) are in the batch; a vision run
    that is not a whole number of blocks leaves its remainder uncompressed in front of the text rows."""
    r = _rng(77)
    n, m, d, H_kv, H_q, R_max, T_cap, N_cap = 12, 5, 8, 2, 4, 5, 9, 64
    N_v = [0, 12, 60, 31, 0, 29]            # blocks 0, 1, 5, 2 (+7 left over), 0, 2 (+5)
    T_own = [4, 0, 1, 2, 0, 0]              # text rows of each sequence (before the left-over vision rows)
    B = len(N_v)
    idx = np.sort(r.choice(n, m, replace=False))
    theta, U = r.normal(size=(H_kv, m, n)), r.normal(size=(H_kv, m, n))
    mu = r.normal(size=(H_kv, d))
    q = r.normal(size=(B, H_q, d))
    K_vis, V_vis = r.normal(size=(B, H_kv, N_cap, d)), r.normal(size=(B, H_kv, N_cap, d))
    for b in range(B):                      # rows a sequence does not have must never be read into a result
        K_vis[b, :, N_v[b]:] = np.nan
        V_vis[b, :, N_v[b]:] = np.nan
    K_t, V_t, R_b, K_tail, V_tail = orc.compress_ragged(np.nan_to_num(K_vis, nan=1e30), np.nan_to_num(V_vis, nan=1e30),
                                                        N_v, idx, U, mu, n, R_max)
    assert list(R_b) == [0, 1, 5, 2, 0, 2] and [k.shape[1] for k in K_tail] == [0, 0, 0, 7, 0, 5]
    K_txt, V_txt = np.full((B, H_kv, T_cap, d), np.nan), np.full((B, H_kv, T_cap, d), np.nan)
    T_b = []
    own = [(r.normal(size=(H_kv, t, d)), r.normal(size=(H_kv, t, d))) for t in T_own]
    for b in range(B):
        t0 = K_tail[b].shape[1]
        K_txt[b, :, :t0], V_txt[b, :, :t0] = K_tail[b], V_tail[b]
        K_txt[b, :, t0:t0 + T_own[b]], V_txt[b, :, t0:t0 + T_own[b]] = own[b]
        T_b.append(t0 + T_own[b])
    K_pad, V_pad = K_t.copy(), V_t.copy()
    for b in range(B):
        K_pad[b, :, R_b[b]:] = np.nan
        V_pad[b, :, R_b[b]:] = np.nan
    got = orc.decode_attend_ragged(q, K_pad, V_pad, theta, U, mu, K_txt, V_txt, R_b, T_b)
    assert np.isfinite(got).all()
    for b in range(B):
        Rb, Tb = int(R_b[b]), T_b[b]
        if Rb == 0 and Tb == 0:
            assert not got[b].any()
            continue
        # the sequence alone: its whole blocks compressed by the uniform function, then the uniform decode forms
        Kb, Vb = orc.compress(K_vis[b:b + 1, :, :Rb * n], V_vis[b:b + 1, :, :Rb * n], idx, U, mu, n)
        assert np.array_equal(Kb[0], K_t[b, :, :Rb]) and np.array_equal(Vb[0], V_t[b, :, :Rb])
        for f in (orc.decode_attend_definition, orc.decode_attend_fused):
            want = f(q[b:b + 1], Kb, Vb, theta, U, mu, K_txt[b:b + 1, :, :Tb], V_txt[b:b + 1, :, :Tb])
            np.testing.assert_allclose(got[b:b + 1], want, atol=1e-11)
        # and against the library routine on the reconstructed blocks + left-over rows + text rows
        K_hat, V_hat = orc.reconstruct(Kb, Vb, theta, U, mu)
        K_all = np.concatenate([K_hat, K_txt[b:b + 1, :, :Tb]], axis=2)
        V_all = np.concatenate([V_hat, V_txt[b:b + 1, :, :Tb]], axis=2)
        np.testing.assert_allclose(got[b:b + 1], _library_attention(q[b:b + 1], K_all, V_all), atol=1e-11)


def test_uniform_lengths_reduce_to_the_uniform_functions():
    p = _problem(31)
    B = p["q"].shape[0]
    K_t, V_t = orc.compress(p["K_vis"], p["V_vis"], p["idx"], p["U"], p["mu"], p["n"])
    want = orc.decode_attend_definition(p["q"], K_t, V_t, p["theta"], p["U"], p["mu"], p["K_txt"], p["V_txt"])
    got = orc.decode_attend_ragged(p["q"], K_t, V_t, p["theta"], p["U"], p["mu"], p["K_txt"], p["V_txt"],
                                   [p["R"]] * B, [p["K_txt"].shape[2]] * B)
    np.testing.assert_allclose(got, want, atol=1e-12)
    K2, V2, R_b, K_tail, V_tail = orc.compress_ragged(p["K_vis"], p["V_vis"], [p["R"] * p["n"]] * B, p["idx"], p["U"],
                                                      p["mu"], p["n"], p["R"])
    assert np.array_equal(K2, K_t) and np.array_equal(V2, V_t) and all(k.shape[1] == 0 for k in K_tail)


# ---------------------------------------------------------------- fused algebra
@pytest.mark.parametrize("seed,kw", [(10, {}), (11, dict(B=1, H_q=4, H_kv=4, R=1, T=0)),
                                     (12, dict(H_q=8, H_kv=1, n=9, m=9, R=2, T=1))])
def test_definition_equals_algorithm_1(seed, kw):
    p = _problem(seed, **kw)
    K_t, V_t = orc.compress(p["K_vis"], p["V_vis"], p["idx"], p["U"], p["mu"], p["n"])
    a = orc.decode_attend_definition(p["q"], K_t, V_t, p["theta"], p["U"], p["mu"], p["K_txt"], p["V_txt"])
    b = orc.decode_attend_fused(p["q"], K_t, V_t, p["theta"], p["U"], p["mu"], p["K_txt"], p["V_txt"])
    np.testing.assert_allclose(a, b, atol=1e-10)


def test_block_order_and_split_merge_invariance():
    # Softmax attention is invariant to permuting KV positions; permuting whole vision
    # blocks must therefore leave the result unchanged, and a log-sum-exp merge of the
    # per-block partial results must reproduce it.
    p = _problem(13)
    K_t, V_t = orc.compress(p["K_vis"], p["V_vis"], p["idx"], p["U"], p["mu"], p["n"])
    ref = orc.decode_attend_definition(p["q"], K_t, V_t, p["theta"], p["U"], p["mu"], p["K_txt"], p["V_txt"])
    perm = [2, 0, 1]
    out = orc.decode_attend_definition(p["q"], K_t[:, :, perm], V_t[:, :, perm], p["theta"], p["U"], p["mu"],
                                       p["K_txt"], p["V_txt"])
    np.testing.assert_allclose(out, ref, atol=1e-12)
    K_hat, V_hat = orc.reconstruct(K_t, V_t, p["theta"], p["U"], p["mu"])
    n, d = p["n"], 8
    parts = [(K_hat[:, :, r * n:(r + 1) * n], V_hat[:, :, r * n:(r + 1) * n]) for r in range(p["R"])]
    parts.append((p["K_txt"], p["V_txt"]))
    B, H_q = p["q"].shape[:2]
    G = H_q // 2
    for b in range(B):
        for hq in range(H_q):
            ms, ls, ys = [], [], []
            for Kp, Vp in parts:
                s = Kp[b, hq // G] @ p["q"][b, hq] / math.sqrt(d)
                ms.append(s.max()); e = np.exp(s - s.max()); ls.append(e.sum()); ys.append(e @ Vp[b, hq // G])
            M = max(ms)
            num = sum(math.exp(mi - M) * yi for mi, yi in zip(ms, ys))
            den = sum(math.exp(mi - M) * li for mi, li in zip(ms, ls))
            np.testing.assert_allclose(num / den, ref[b, hq], atol=1e-12)


# ---------------------------------------------------------------- brute force, tiny grid
def test_tiny_grid_brute_force():
    """n = 4 (2x2 grid), m = 2, d = 2, G = 1, T = 1: every step with scalar loops."""
    r = _rng(14)
    n, m, d, T = 4, 2, 2, 1
    K = r.standard_normal((n, d)); V = r.standard_normal((n, d))
    kt = r.standard_normal((T, d)); vt = r.standard_normal((T, d))
    q = r.standard_normal(d)
    th = r.standard_normal((m, n)); U = r.standard_normal((m, n)); mu = r.standard_normal(d)
    idx = [1, 3]
    # compress
    Kc = [[K[idx[j]][c] for c in range(d)] for j in range(m)]
    Vc = [[sum(U[j][i] * (V[i][c] - mu[c]) for i in range(n)) for c in range(d)] for j in range(m)]
    # reconstruct
    Kh = [[sum(th[j][i] * Kc[j][c] for j in range(m)) for c in range(d)] for i in range(n)]
    Vh = [[sum(U[j][i] * Vc[j][c] for j in range(m)) + mu[c] for c in range(d)] for i in range(n)]
    rowsK = Kh + [list(kt[0])]
    rowsV = Vh + [list(vt[0])]
    logits = [sum(q[c] * rk[c] for c in range(d)) / math.sqrt(d) for rk in rowsK]
    mx = max(logits)
    ex = [math.exp(l - mx) for l in logits]
    Z = sum(ex)
    want = [sum(ex[i] / Z * rowsV[i][c] for i in range(n + T)) for c in range(d)]

    K_t, V_t = orc.compress(K[None, None], V[None, None], np.array(idx), U[None], mu[None], n)
    np.testing.assert_allclose(K_t[0, 0, 0], np.array(Kc), atol=0)
    np.testing.assert_allclose(V_t[0, 0, 0], np.array(Vc), atol=1e-14)
    for f in (orc.decode_attend_definition, orc.decode_attend_fused):
        got = f(q[None, None], K_t, V_t, th[None], U[None], mu[None], kt[None, None], vt[None, None])
        np.testing.assert_allclose(got[0, 0], want, atol=1e-13)


def test_two_heads_two_blocks_brute_force():
    """G = 2 query heads per KV head, H_kv = 2, R = 2 blocks, T = 2 text rows, per-head index sets: every step with
    scalar loops over plain Python lists, so that the head map hq -> hq // G, the block offsets r*n + i and the
    per-head parameters are all written out independently of the oracle's array code."""
    r = _rng(15)
    B, H_kv, G, R, n, m, d, T = 1, 2, 2, 2, 3, 2, 2, 2
    H_q = H_kv * G
    K = r.standard_normal((B, H_kv, R * n, d)); V = r.standard_normal((B, H_kv, R * n, d))
    Kx = r.standard_normal((B, H_kv, T, d)); Vx = r.standard_normal((B, H_kv, T, d))
    q = r.standard_normal((B, H_q, d))
    th = r.standard_normal((H_kv, m, n)); U = r.standard_normal((H_kv, m, n)); mu = r.standard_normal((H_kv, d))
    idx = [[0, 2], [1, 2]]
    want = [[0.0] * d for _ in range(H_q)]
    for hq in range(H_q):
        h = hq // G
        rowsK, rowsV = [], []
        for blk in range(R):
            Kc = [[K[0][h][blk * n + idx[h][j]][c] for c in range(d)] for j in range(m)]
            Vc = [[sum(U[h][j][i] * (V[0][h][blk * n + i][c] - mu[h][c]) for i in range(n)) for c in range(d)] for j in range(m)]
            for i in range(n):
                rowsK.append([sum(th[h][j][i] * Kc[j][c] for j in range(m)) for c in range(d)])
                rowsV.append([sum(U[h][j][i] * Vc[j][c] for j in range(m)) + mu[h][c] for c in range(d)])
        for t in range(T):
            rowsK.append([Kx[0][h][t][c] for c in range(d)])
            rowsV.append([Vx[0][h][t][c] for c in range(d)])
        logits = [sum(q[0][hq][c] * rk[c] for c in range(d)) / math.sqrt(d) for rk in rowsK]
        mx = max(logits)
        ex = [math.exp(l - mx) for l in logits]
        Z = sum(ex)
        want[hq] = [sum(ex[i] / Z * rowsV[i][c] for i in range(len(rowsV))) for c in range(d)]
    K_t, V_t = orc.compress(K, V, np.array(idx), U, mu, n)
    for f in (orc.decode_attend_definition, orc.decode_attend_fused):
        got = f(q, K_t, V_t, th, U, mu, Kx, Vx)
        np.testing.assert_allclose(got[0], np.array(want), atol=1e-13)


def test_scalar_closed_form():
    """n = 2, m = 1, d = 1: the whole path is a three-way logistic mixture in closed form."""
    k0, k1, v0, v1 = 0.7, -0.4, 1.5, -2.0
    a, b, u0, u1, mu, q, kt, vt = 0.9, -0.3, 0.6, 0.8, 0.25, 1.3, 0.2, 3.0
    K = np.array([k0, k1]).reshape(1, 1, 2, 1); V = np.array([v0, v1]).reshape(1, 1, 2, 1)
    K_t, V_t = orc.compress(K, V, np.array([0]), np.array([[[u0, u1]]]), np.array([[mu]]), 2)
    vtil = u0 * (v0 - mu) + u1 * (v1 - mu)
    assert K_t[0, 0, 0, 0, 0] == k0 and abs(V_t[0, 0, 0, 0, 0] - vtil) < 1e-15
    l = [q * a * k0, q * b * k0, q * kt]                     # sigma = 1/sqrt(1)
    w = [math.exp(x) for x in l]
    want = (w[0] * (u0 * vtil + mu) + w[1] * (u1 * vtil + mu) + w[2] * vt) / sum(w)
    for f in (orc.decode_attend_definition, orc.decode_attend_fused):
        got = f(np.array([[[q]]]), K_t, V_t, np.array([[[a, b]]]), np.array([[[u0, u1]]]), np.array([[mu]]),
                np.array([[[[kt]]]]), np.array([[[[vt]]]]))
        assert abs(got[0, 0, 0] - want) < 1e-14


# ---------------------------------------------------------------- factored key reconstructor
def test_collapsed_two_layer_reconstructor():
    """theta = W1 W2: (i) with k = m and W1 = I it is W2 itself; (ii) the keys reconstructed layer by layer with scalar
    loops (first the k hidden rows, then the n positions) are theta^T K_tilde; (iii) its rank is at most k; (iv) a decode
    step with the collapsed theta equals one whose scores are expanded in two skinny steps, (S W1) W2."""
    r = _rng(31)
    H, m, k, n, d = 2, 5, 3, 7, 4
    W1 = r.standard_normal((H, m, k)); W2 = r.standard_normal((H, k, n))
    th = orc.collapse_reconstructor(W1, W2)
    eye = np.broadcast_to(np.eye(m), (H, m, m))
    W2m = r.standard_normal((H, m, n))
    assert np.array_equal(orc.collapse_reconstructor(eye, W2m), W2m)
    Kt = r.standard_normal((m, d))
    for h in range(H):
        hidden = [[sum(W1[h][j][l] * Kt[j][c] for j in range(m)) for c in range(d)] for l in range(k)]
        Kh = [[sum(W2[h][l][i] * hidden[l][c] for l in range(k)) for c in range(d)] for i in range(n)]
        np.testing.assert_allclose(th[h].T @ Kt, np.array(Kh), atol=1e-13)
        assert np.linalg.matrix_rank(th[h]) <= k
    # (iv): Alg. 1 with L = (S W1) W2 taken in two steps, one head, one block, no text
    q = r.standard_normal(d); V = r.standard_normal((n, d)); U = r.standard_normal((1, m, n)); mu = r.standard_normal((1, d))
    K_t = Kt[None, None, None]; V_t = (U[0] @ (V - mu[0]))[None, None, None]
    S = Kt @ q / math.sqrt(d)
    L = (S @ W1[0]) @ W2[0]
    P = np.exp(L - L.max()); P /= P.sum()
    want = (P @ U[0].T) @ V_t[0, 0, 0] + P.sum() * mu[0]
    got = orc.decode_attend_fused(q[None, None], K_t, V_t, th[:1], U, mu, np.zeros((1, 1, 0, d)), np.zeros((1, 1, 0, d)))
    np.testing.assert_allclose(got[0, 0], want, atol=1e-13)


# ---------------------------------------------------------------- sizes (App. D)
def _golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                vals[k] = float(v)
    return vals


def test_memory_footprint_hand_written_integers():
    """App. D Eq. 2 on sizes small enough to count by hand (bytes): B = 1, H_kv = 1, one block of n = 4 tokens kept at
    m = 2 (rho = 0.5), d = 2, 2-byte elements, c = 1 prompt token, t = 1 generated token.
      compressed cache : K and V, (1 + 2 + 1) tokens x 2 channels x 2 bytes      = 2 * 16 = 32
      S_recon(theta)   : 1 head x 2 x 4 entries x 2 bytes                         = 16
      S_PCA(U, mu)     : U 1 x 2 x 4 x 2 bytes = 16, mu 1 x 2 x 2 bytes = 4        = 20
    and Eq. 1 for the same sequence: (1 + 4 + 1) tokens x 2 x 2 bytes, K and V    = 48."""
    assert orc.footprint_kvcapsule(1, 1, 1, 4, 1, 1, 2, 2, 500) == 32 + 16 + 20 == 68
    assert orc.footprint_base(1, 1, 1, 4, 1, 2, 2) == 48
    # three blocks, two KV heads, batch 3, 4-byte parameters beside 2-byte cache entries:
    #   cache 2 * 3 * 2 * (1 + 3*2 + 1) * 2 * 2 = 384;  theta 2*2*4*4 = 64;  U 64 + mu 2*2*4 = 16
    assert orc.footprint_kvcapsule(3, 2, 1, 4, 3, 1, 2, 2, 500, b_param=4) == 384 + 64 + 80 == 528
    # the parameter terms do not grow with the batch (Sec. 4.3): only the cache term does
    assert orc.footprint_kvcapsule(6, 2, 1, 4, 3, 1, 2, 2, 500, b_param=4) == 768 + 144


def test_memory_footprint_closed_forms_and_paper_ratio():
    g = _golden("paper_constants.txt")
    B, H_kv, d, b = 16, 4, 128, 2
    n, R, c, t = 1024, 8, 256, 0
    m = orc.retained_len(n, 600)
    base = orc.footprint_base(B, H_kv, c, R * n, t, d, b)
    ours = orc.footprint_kvcapsule(B, H_kv, c, n, R, t, d, b, 600)
    assert base == 2 * 16 * 4 * (256 + 8192) * 128 * 2
    cache = 2 * B * H_kv * (c + R * m + t) * d * b
    assert ours == cache + 2 * H_kv * m * n * b + H_kv * d * b
    # the paper's headline persistent-memory reduction at 60 % compression
    assert round(base / cache, 1) == g["memory_reduction_at_60pct"]
    # with the batch-independent parameter overhead included the reduction is a little lower
    assert 2.2 < base / ours < base / cache
    # vision-only reduction is 1 / l_r up to the ceiling
    for nn in (576, 1024, 256):
        assert abs(nn / orc.retained_len(nn, 600) - 2.5) < 0.02
    # parameter overhead is independent of batch size and generated length (Sec. 4.3)
    o1 = orc.footprint_kvcapsule(1, H_kv, c, n, R, 0, d, b, 600) - 2 * 1 * H_kv * (c + R * m) * d * b
    o2 = orc.footprint_kvcapsule(64, H_kv, c, n, R, 99, d, b, 600) - 2 * 64 * H_kv * (c + R * m + 99) * d * b
    assert o1 == o2
