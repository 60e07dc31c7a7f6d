"""CPU pins of the fp64 oracle: each test checks it against something other than itself --
brute-force masked attention, closed forms, reductions to textbook attention, an independent
transcription of Algorithm 1, finite differences, and gradient identities."""
import os

import numpy as np
import pytest

import oracle
from oracle.chunked import attend_chunked
from tests.brute import bf16_bits_to_f64, f64_to_bf16_bits, layer_brute

RNG = np.random.default_rng(1234)


def rand_bf16(shape, rng=RNG, scale=1.0):
    return f64_to_bf16_bits(rng.standard_normal(shape) * scale)


def make(B, Lq, Hq, Hkv, D, Lk=None, rng=RNG, density=0.4):
    Lk = Lq if Lk is None else Lk
    Q = rand_bf16((B, Lq, Hq, D), rng)
    K = rand_bf16((B, Lk, Hkv, D), rng)
    V = rand_bf16((B, Lk, Hkv, D), rng)
    d = (rng.random((B, Lq)) < density).astype(np.uint8)
    return Q, K, V, d


# ---------------------------------------------------------------- routing and compaction (Eq. 3, Sec. 3.2)

def test_route_threshold_ties_and_specials():
    # Eq. 3 uses >=; a zero-initialised router (logit 0, sigmoid 0.5) must route every token.
    lines = [l.split() for l in open(os.path.join(os.path.dirname(__file__), "golden", "router_tie.txt"))
             if l.strip() and not l.startswith("#")]
    z = np.array([float(a) for a, _ in lines], np.float32)
    want = np.array([int(b) for _, b in lines], np.uint8)
    assert np.array_equal(oracle.route(z, 0.0), want)
    assert oracle.route(np.zeros(16, np.float32), 0.0).all()


def test_compact_matches_loop():
    rng = np.random.default_rng(7)
    for B, L, rho in [(1, 1, 1.0), (1, 1, 0.0), (2, 37, 0.3), (3, 257, 0.9), (1, 1000, 0.01)]:
        d = (rng.random((B, L)) < rho).astype(np.uint8)
        q_idx, n, prefix = oracle.compact(d)
        for b in range(B):
            pos = [t for t in range(L) if d[b, t]]
            assert n[b] == len(pos)
            assert list(q_idx[b, :len(pos)]) == pos
            assert (q_idx[b, len(pos):] == -1).all()
            assert list(prefix[b]) == [sum(d[b, :t]) for t in range(L + 1)]


# ---------------------------------------------------------------- forward definition vs brute force

@pytest.mark.parametrize("B,Lq,Lk,Hq,Hkv,D,W", [
    (1, 33, 33, 1, 1, 8, 5),
    (2, 48, 48, 4, 2, 16, 7),
    (1, 20, 64, 6, 2, 8, 9),      # Lk > Lq: bottom-right aligned positions
    (1, 40, 40, 2, 1, 4, 0),      # W = 0: self only
    (1, 40, 40, 2, 2, 4, 100),    # W >= L - 1: local == full causal
])
def test_forward_matches_bruteforce_masks(B, Lq, Lk, Hq, Hkv, D, W):
    Q, K, V, d = make(B, Lq, Hq, Hkv, D, Lk)
    sh = oracle.Shape(B, Lq, Lk, Hq, Hkv, D, W)
    got = oracle.forward_full(sh, Q, K, V, d)
    ref = layer_brute(bf16_bits_to_f64(Q), bf16_bits_to_f64(K), bf16_bits_to_f64(V), d, W)
    for k in ("s", "a", "o", "lse_loc"):
        np.testing.assert_allclose(got[k], ref[k], rtol=0, atol=1e-12, err_msg=k)
    on = np.broadcast_to(d[:, None, :].astype(bool), got["lse_glb"].shape)
    np.testing.assert_allclose(got["lse_glb"][on], ref["lse_glb"][on], rtol=0, atol=1e-12)
    assert np.isnan(got["lse_glb"][~on]).all()
    assert (got["a"][~d.astype(bool)] == 0).all()          # a_t = 0 when d_t = 0 (Eq. 4)


def test_custom_scale_and_offset():
    Q, K, V, d = make(1, 16, 2, 1, 8, 24)
    sh = oracle.Shape(1, 16, 24, 2, 1, 8, 6, q_pos_offset=3, scale=0.37)
    got = oracle.forward_full(sh, Q, K, V, d)
    ref = layer_brute(bf16_bits_to_f64(Q), bf16_bits_to_f64(K), bf16_bits_to_f64(V), d, 6, scale=0.37, offset=3)
    np.testing.assert_allclose(got["o"], ref["o"], rtol=0, atol=1e-12)


def test_running_softmax_over_any_chunking_equals_definition():
    # Algorithm 1's evaluation order (key chunks, carried maximum / sum / values, early stop at the chunk of the
    # group's last position) for uniform, ragged and random chunkings and row groupings, against the two-pass oracle
    rng = np.random.default_rng(5)
    for n, D, rows_per_group, chunking, rho in [(37, 8, 4, 4, 0.5), (64, 4, 4, 8, 0.2), (50, 8, 7, 5, 1.0),
                                                (30, 8, 4, 4, 0.05), (61, 8, 5, "random", 0.4), (48, 4, 48, 1, 0.3)]:
        Q, K, V, d = make(1, n, 1, 1, D, rng=rng, density=rho)
        d[0, 3] = 1
        W = 4
        got = oracle.forward_full(oracle.Shape(1, n, n, 1, 1, D, W), Q, K, V, d)
        q_idx, n_c, _ = oracle.compact(d)
        idx = q_idx[0, :n_c[0]]
        q, k, v = (bf16_bits_to_f64(x)[0, :, 0] for x in (Q, K, V))
        if chunking == "random":
            cuts = np.sort(rng.choice(np.arange(1, n), size=9, replace=False))
            bounds = [0, *cuts.tolist(), n]
        else:
            bounds = list(range(0, n, chunking)) + [n]
        for g0 in range(0, len(idx), rows_per_group):       # routed rows, grouped as a compact tile would be
            rows = idx[g0:g0 + rows_per_group]
            out, lse, visited = attend_chunked(q[rows], k, v, rows, bounds)
            np.testing.assert_allclose(out, got["a"][0, rows, 0], rtol=0, atol=1e-12)
            np.testing.assert_allclose(lse, got["lse_glb"][0, 0, rows], rtol=0, atol=1e-12)
            assert visited == np.searchsorted(bounds, rows.max(), side="right")    # no chunk after the last position
        for g0 in range(0, n, rows_per_group):              # all rows with the window bound: the local module
            rows = np.arange(g0, min(g0 + rows_per_group, n))
            out, lse, _ = attend_chunked(q[rows], k, v, rows, bounds, lowest=rows - W)
            np.testing.assert_allclose(out, got["s"][0, rows, 0], rtol=0, atol=1e-12)
            np.testing.assert_allclose(lse, got["lse_loc"][0, 0, rows], rtol=0, atol=1e-12)


# ---------------------------------------------------------------- closed forms

def test_zero_keys_gives_window_and_prefix_means():
    # K == 0 -> uniform soft-max: s_t = mean of v over the last min(t, W) + 1 keys (pins "W + 1 keys"),
    # a_t = prefix mean; lse = log(count).
    B, L, Hq, Hkv, D, W = 1, 300, 2, 1, 4, 17
    Q, _, V, d = make(B, L, Hq, Hkv, D)
    K = np.zeros((B, L, Hkv, D), np.uint16)
    got = oracle.forward_full(oracle.Shape(B, L, L, Hq, Hkv, D, W), Q, K, V, d)
    v = bf16_bits_to_f64(V)[0, :, 0]
    cs = np.concatenate([np.zeros((1, D)), np.cumsum(v, axis=0)])
    t = np.arange(L)
    lo = np.maximum(0, t - W)
    cnt = t - lo + 1
    s_ref = (cs[t + 1] - cs[lo]) / cnt[:, None]
    a_ref = cs[t + 1] / (t + 1)[:, None]
    for h in range(Hq):
        np.testing.assert_allclose(got["s"][0, :, h], s_ref, atol=1e-12)
        np.testing.assert_allclose(got["lse_loc"][0, h], np.log(np.minimum(t + 1, W + 1)), atol=1e-12)
        on = d[0].astype(bool)
        np.testing.assert_allclose(got["a"][0, on, h], a_ref[on], atol=1e-12)
        np.testing.assert_allclose(got["lse_glb"][0, h, on], np.log(t + 1)[on], atol=1e-12)


def test_constant_values_give_one_plus_d():
    B, L, Hq, Hkv, D, W = 1, 64, 2, 2, 8, 9
    Q, K, _, d = make(B, L, Hq, Hkv, D)
    c = f64_to_bf16_bits(np.linspace(-2, 2, D))
    V = np.broadcast_to(c, (B, L, Hkv, D)).copy()
    got = oracle.forward_full(oracle.Shape(B, L, L, Hq, Hkv, D, W), Q, K, V, d)
    want = (1 + d[0])[:, None, None] * bf16_bits_to_f64(c)[None, None, :]
    np.testing.assert_allclose(got["o"][0], np.broadcast_to(want, got["o"][0].shape), atol=1e-12)


def test_dominant_key_selects_its_value():
    L, D, W = 40, 8, 4
    Q = np.zeros((1, L, 1, D)); K = np.zeros((1, L, 1, D))
    Q[..., 0] = 64.0
    K[0, 10, 0, 0] = 64.0                  # key 10 scores 64*64/sqrt(8) above everything else
    Q, K = f64_to_bf16_bits(Q), f64_to_bf16_bits(K)
    V = rand_bf16((1, L, 1, D))
    d = np.ones((1, L), np.uint8)
    got = oracle.forward_full(oracle.Shape(1, L, L, 1, 1, D, W), Q, K, V, d)
    v = bf16_bits_to_f64(V)[0, :, 0]
    np.testing.assert_allclose(got["a"][0, 10:, 0], np.broadcast_to(v[10], (L - 10, D)), atol=1e-9)
    np.testing.assert_allclose(got["s"][0, 10:15, 0], np.broadcast_to(v[10], (5, D)), atol=1e-9)  # 10 inside window for t <= 14
    assert np.abs(got["s"][0, 15, 0] - v[10]).max() > 1e-3                                         # and outside at t = 15


# ---------------------------------------------------------------- reductions to textbook attention

def _softmax_attention(q, k, v, allowed, scale):
    out = np.zeros_like(q)
    for i in range(q.shape[0]):
        js = [j for j in range(k.shape[0]) if allowed(i, j)]
        sc = np.array([scale * float(q[i] @ k[j]) for j in js])
        w = np.exp(sc - sc.max()); w /= w.sum()
        out[i] = sum(w[n] * v[j] for n, j in enumerate(js))
    return out


def test_reductions():
    B, L, D, W = 1, 24, 4, 5
    Q, K, V, _ = make(B, L, 1, 1, D)
    q, k, v = (bf16_bits_to_f64(x)[0, :, 0] for x in (Q, K, V))
    sc = 1 / np.sqrt(D)
    full = _softmax_attention(q, k, v, lambda i, j: j <= i, sc)
    swa = _softmax_attention(q, k, v, lambda i, j: 0 <= i - j <= W, sc)
    zeros, ones = np.zeros((B, L), np.uint8), np.ones((B, L), np.uint8)
    # d == 0 -> O is sliding-window attention
    g = oracle.forward_full(oracle.Shape(B, L, L, 1, 1, D, W), Q, K, V, zeros)
    np.testing.assert_allclose(g["o"][0, :, 0], swa, atol=1e-12)
    # d == 1 -> A is full causal attention, O = S + A
    g = oracle.forward_full(oracle.Shape(B, L, L, 1, 1, D, W), Q, K, V, ones)
    np.testing.assert_allclose(g["a"][0, :, 0], full, atol=1e-12)
    np.testing.assert_allclose(g["o"][0, :, 0], swa + full, atol=1e-12)
    # W >= L - 1 -> S is full causal attention; with d == 1 and one Q/K/V set, O = 2 * full
    g = oracle.forward_full(oracle.Shape(B, L, L, 1, 1, D, L - 1), Q, K, V, ones)
    np.testing.assert_allclose(g["s"][0, :, 0], full, atol=1e-12)
    np.testing.assert_allclose(g["o"][0, :, 0], 2 * full, atol=1e-12)
    # W == 0 -> S = V
    g = oracle.forward_full(oracle.Shape(B, L, L, 1, 1, D, 0), Q, K, V, zeros)
    np.testing.assert_allclose(g["s"][0, :, 0], v, atol=1e-12)


# ---------------------------------------------------------------- backward

def _loss_f64(sh, Q, K, V, d, dO):
    with oracle.f64_inputs():
        return float((oracle.forward_full(sh, Q, K, V, d)["o"] * dO).sum())


def test_backward_matches_finite_differences():
    rng = np.random.default_rng(11)
    B, L, Hq, Hkv, D, W = 1, 16, 2, 1, 8, 3
    Q, K, V, dO = (rng.standard_normal(s) for s in [(B, L, Hq, D), (B, L, Hkv, D), (B, L, Hkv, D), (B, L, Hq, D)])
    d = (rng.random((B, L)) < 0.5).astype(np.uint8)
    d[0, 0] = 1
    sh = oracle.Shape(B, L, L, Hq, Hkv, D, W)
    with oracle.f64_inputs():
        dQ, dK, dV = oracle.backward_full(sh, Q, K, V, d, dO)
    h = 1e-6
    for name, X, G in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        flat = X.reshape(-1)
        idx = rng.choice(flat.size, 40, replace=False)
        for i in idx:
            old = flat[i]
            flat[i] = old + h; lp = _loss_f64(sh, Q, K, V, d, dO)
            flat[i] = old - h; lm = _loss_f64(sh, Q, K, V, d, dO)
            flat[i] = old
            fd = (lp - lm) / (2 * h)
            assert abs(fd - G.reshape(-1)[i]) <= 1e-7 * max(1.0, abs(fd)), (name, i, fd, G.reshape(-1)[i])


def test_backward_identities():
    B, L, Hq, Hkv, D, W = 2, 40, 4, 2, 8, 6
    Q, K, V, d = make(B, L, Hq, Hkv, D)
    dO = rand_bf16((B, L, Hq, D))
    sh = oracle.Shape(B, L, L, Hq, Hkv, D, W)
    dQ, dK, dV = oracle.backward_full(sh, Q, K, V, d, dO)
    # every soft-max row sums to one -> sum_j dV_j = sum_t (1 + d_t) dO_t over the group's heads
    g = bf16_bits_to_f64(dO) * (1 + d)[:, :, None, None]
    want = g.reshape(B, L, Hkv, Hq // Hkv, D).sum(axis=(1, 3))
    np.testing.assert_allclose(dV.sum(axis=1), want, atol=1e-10)
    # V == const -> outputs do not depend on Q, K
    c = f64_to_bf16_bits(np.linspace(-1, 1, D))
    Vc = np.broadcast_to(c, V.shape).copy()
    dQc, dKc, _ = oracle.backward_full(sh, Q, K, Vc, d, dO)
    assert np.abs(dQc).max() < 1e-12 and np.abs(dKc).max() < 1e-12
    # non-routed rows receive the local term only: equal to a d == 0 run on those rows
    dQ0, _, _ = oracle.backward_full(sh, Q, K, V, np.zeros_like(d), dO)
    off = ~d.astype(bool)
    np.testing.assert_allclose(dQ[off], dQ0[off], atol=1e-13)
    assert np.abs(dQ[~off] - dQ0[~off]).max() > 1e-3


def test_sampled_backward_modes_equal_full():
    B, L, Hq, Hkv, D, W = 2, 48, 4, 2, 8, 7
    Q, K, V, d = make(B, L, Hq, Hkv, D)
    dO = rand_bf16((B, L, Hq, D))
    sh = oracle.Shape(B, L, L, Hq, Hkv, D, W)
    dQ, dK, dV = oracle.backward_full(sh, Q, K, V, d, dO)
    rb = np.array([0, 1, 1, 0]); rh = np.array([0, 3, 2, 1]); rt = np.array([0, 47, 13, 30])
    np.testing.assert_allclose(oracle.dq_rows(sh, Q, K, V, d, dO, rb, rh, rt), dQ[rb, rt, rh], atol=1e-12)
    js = np.array([0, 5, 5, 47, 20])
    for b, g in [(0, 0), (1, 1)]:
        dk, dv = oracle.dkv_cols(sh, Q, K, V, d, dO, b, g, js)
        np.testing.assert_allclose(dk, dK[b, js, g], atol=1e-12)
        np.testing.assert_allclose(dv, dV[b, js, g], atol=1e-12)


def test_dgate_matches_definition():
    # Eq. 7, first term: (dL/do_t)^T a_t, a_t taken for every token
    B, L, Hq, Hkv, D, W = 1, 20, 2, 1, 4, 3
    Q, K, V, _ = make(B, L, Hq, Hkv, D)
    dO = rand_bf16((B, L, Hq, D))
    sh = oracle.Shape(B, L, L, Hq, Hkv, D, W)
    ref = layer_brute(bf16_bits_to_f64(Q), bf16_bits_to_f64(K), bf16_bits_to_f64(V), np.ones((B, L), np.uint8), W)
    want = (ref["a"] * bf16_bits_to_f64(dO)).sum(axis=(2, 3))[0]
    got = oracle.dgate_rows(sh, Q, K, V, dO, np.zeros(L, np.int32), np.arange(L))
    np.testing.assert_allclose(got, want, atol=1e-12)


def test_router_logits_closed_forms():
    # a one-hot router weight picks one coordinate of s_t; a zero router gives the bias for every token, and a
    # zero-initialised router (bias 0) sits exactly on the threshold, which routes every token (Section 3.1)
    B, L, Hq, D = 2, 9, 2, 4
    S = rand_bf16((B, L, Hq, D))
    s = bf16_bits_to_f64(S).reshape(B, L, Hq * D)
    w = np.zeros(Hq * D); w[5] = 2.0
    np.testing.assert_allclose(oracle.router_logits(S, w, 0.25), 2.0 * s[:, :, 5] + 0.25, atol=1e-15)
    z0 = oracle.router_logits(S, np.zeros(Hq * D), 0.0)
    assert (z0 == 0).all() and oracle.route(z0.astype(np.float32), 0.0).all()
    np.testing.assert_allclose(oracle.gate_regulariser_sum(z0), np.full(B, L * 0.25), atol=1e-15)   # sigmoid(0)^2 = 1/4


def test_gate_regulariser_closed_forms():
    # Eq. 6 without its lambda / (n L) factor: sum over tokens of sigmoid(z_t)^2.  sigmoid(ln 3) = 3/4 and
    # sigmoid(-ln 3) = 1/4, so the squares are 9/16 and 1/16: a sign slip in the exponent, a missing square or a sum over the
    # wrong axis fails.
    ln3 = np.log(3.0)
    z = np.array([[ln3, ln3, -ln3], [-ln3, -ln3, -ln3]])
    np.testing.assert_allclose(oracle.gate_regulariser_sum(z), [2 * 0.5625 + 0.0625, 3 * 0.0625], rtol=1e-14)
    np.testing.assert_allclose(oracle.gate_regulariser_sum(np.array([[40.0, -40.0]])), [1.0], rtol=1e-14)


def test_router_backward_is_the_gradient_of_the_relaxed_loss():
    # Under the straight-through estimator the loss seen by the router is, with a_t and dL/do_t held fixed,
    #   F(W, bias, s) = sum_t g_t * sigmoid(z_t) + c * sum_t sigmoid(z_t)^2,   z_t = W s_t + bias,  g_t = dL/do_t . a_t
    # (Eq. 5 with d_t -> d_hat_t, plus the regulariser of Eq. 6).  Central differences of F pin dW, dbias and the
    # router's contribution to dL/ds_t: a dropped factor 2, a missing sigmoid derivative or a wrong sign fails.
    B, L, Hq, D = 2, 7, 2, 4
    rng = np.random.default_rng(17)
    S = rand_bf16((B, L, Hq, D))
    s = bf16_bits_to_f64(S).reshape(B, L, Hq * D)
    w = rng.standard_normal(Hq * D) * 0.4
    bias, c = -0.2, 0.37
    g = rng.standard_normal((B, L))

    def F(w_, bias_, s_):
        d_hat = 1.0 / (1.0 + np.exp(-(s_ @ w_ + bias_)))
        return float((g * d_hat).sum() + c * (d_hat ** 2).sum())

    z = oracle.router_logits(S, w, bias)
    dO = rand_bf16((B, L, Hq, D))
    dz, dw, dbias, dS = oracle.router_backward(S, w, z, g, c, dO)
    eps = 1e-6
    for k in range(Hq * D):
        e = np.zeros(Hq * D); e[k] = eps
        assert abs((F(w + e, bias, s) - F(w - e, bias, s)) / (2 * eps) - dw[k]) < 1e-7
    assert abs((F(w, bias + eps, s) - F(w, bias - eps, s)) / (2 * eps) - dbias) < 1e-7
    ds_router = dS.reshape(B, L, Hq * D) - bf16_bits_to_f64(dO).reshape(B, L, Hq * D)
    for (b, t, k) in [(0, 0, 0), (1, 3, 5), (1, 6, 7)]:
        sp, sm = s.copy(), s.copy()
        sp[b, t, k] += eps; sm[b, t, k] -= eps
        assert abs((F(w, bias, sp) - F(w, bias, sm)) / (2 * eps) - ds_router[b, t, k]) < 1e-7
    # closed form on the threshold: z = 0 gives d_hat = 1/2, so dz = (g + c) / 4
    dz0, _, _, _ = oracle.router_backward(S, w, np.zeros((B, L)), g, c)
    np.testing.assert_allclose(dz0, (g + c) / 4.0, atol=1e-15)
