"""The algebra behind L2A_FLAG_SHARED_WINDOW, checked in fp64 against the oracle's plain definition (no GPU).

With one Q/K/V set for both modules, a routed row's soft-max over the whole prefix splits into the keys before its
window and the window itself (which the local module has already reduced):
  a_t = (e^{lse_out} o_out + e^{lse_loc} s_t) / (e^{lse_out} + e^{lse_loc}),  lse_glb = log(e^{lse_out} + e^{lse_loc}),
and in the backward the window's share of the global gradient rides on the local pairs with
  P' = (1 + beta) P_loc,  Delta' = (Delta_loc + beta Delta_glb) / (1 + beta),  beta = e^{lse_loc - lse_glb},
while the global pairs stop before the window.  Both must reproduce Eq. 2-5 and their VJP exactly."""
import numpy as np
import pytest

import oracle


def _inputs(B, Lq, Lk, Hq, Hkv, D, seed):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((B, Lq, Hq, D)), rng.standard_normal((B, Lk, Hkv, D)),
            rng.standard_normal((B, Lk, Hkv, D)), rng.standard_normal((B, Lq, Hq, D)))


@pytest.mark.parametrize("B,Lq,Lk,Hq,Hkv,D,W,rho", [(1, 37, 37, 2, 1, 8, 5, 0.5), (2, 20, 33, 4, 2, 4, 0, 0.6),
                                                   (1, 25, 25, 1, 1, 8, 40, 1.0), (1, 30, 30, 2, 2, 4, 7, 0.0)])
def test_split_softmax_and_merged_statistics_reproduce_the_layer(B, Lq, Lk, Hq, Hkv, D, W, rho):
    Q, K, V, dO = _inputs(B, Lq, Lk, Hq, Hkv, D, seed=Lq + W)
    d = (np.random.default_rng(W + 1).random((B, Lq)) < rho).astype(np.uint8)
    sh = oracle.Shape(B, Lq, Lk, Hq, Hkv, D, W)
    with oracle.f64_inputs():
        ref = oracle.forward_full(sh, Q, K, V, d)
        dQ_ref, dK_ref, dV_ref = oracle.backward_full(sh, Q, K, V, d, dO)
    off, G, scale = Lk - Lq, Hq // Hkv, 1.0 / np.sqrt(D)
    o = np.zeros_like(Q)
    a_all = np.zeros_like(Q)
    lse_glb = np.full((B, Hq, Lq), np.nan)
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)
    for b in range(B):
        for h in range(Hq):
            g = h // G
            for t in range(Lq):
                p = t + off
                lo = max(0, p - W)
                z = scale * (K[b, :p + 1, g] @ Q[b, t, h])          # scores against the causal prefix
                zw, zo = z[lo:], z[:lo]                             # window | keys before it
                lse_loc = np.log(np.exp(zw - zw.max()).sum()) + zw.max()
                P_loc = np.exp(zw - lse_loc)
                s = P_loc @ V[b, lo:p + 1, g]
                assert np.allclose(s, ref["s"][b, t, h]) and np.isclose(lse_loc, ref["lse_loc"][b, h, t])
                o[b, t, h] = s
                d_loc = dO[b, t, h] @ s                             # Delta of the local module
                dP_w = V[b, lo:p + 1, g] @ dO[b, t, h]              # dP = dO V^T, common to both modules
                P_w = P_loc                                        # what the local pairs use as P
                if not d[b, t]:
                    dS_w = P_loc * (dP_w - d_loc)
                else:
                    if lo > 0:
                        lse_out = np.log(np.exp(zo - zo.max()).sum()) + zo.max()
                        o_out = np.exp(zo - lse_out) @ V[b, :lo, g]
                    else:
                        lse_out, o_out = -np.inf, np.zeros(D)
                    m = max(lse_out, lse_loc)
                    w_out, w_loc = np.exp(lse_out - m), np.exp(lse_loc - m)
                    a = (w_out * o_out + w_loc * s) / (w_out + w_loc)
                    lg = m + np.log(w_out + w_loc)
                    assert np.allclose(a, ref["a"][b, t, h]) and np.isclose(lg, ref["lse_glb"][b, h, t])
                    a_all[b, t, h], lse_glb[b, h, t] = a, lg
                    o[b, t, h] = s + a
                    d_glb = dO[b, t, h] @ a
                    beta = np.exp(lse_loc - lg)
                    # the window, carried by the local pairs with merged statistics
                    P_w = np.exp(zw - (lse_loc - np.log1p(beta)))      # = (1 + beta) P_loc
                    d1 = (d_loc + beta * d_glb) / (1.0 + beta)
                    dS_w = P_w * (dP_w - d1)
                    # the keys before the window, by the global pairs
                    if lo > 0:
                        P_o = np.exp(zo - lg)
                        dS_o = P_o * (V[b, :lo, g] @ dO[b, t, h] - d_glb)
                        dQ[b, t, h] += scale * (dS_o @ K[b, :lo, g])
                        dK[b, :lo, g] += scale * np.outer(dS_o, Q[b, t, h])
                        dV[b, :lo, g] += np.outer(P_o, dO[b, t, h])
                dQ[b, t, h] += scale * (dS_w @ K[b, lo:p + 1, g])
                dK[b, lo:p + 1, g] += scale * np.outer(dS_w, Q[b, t, h])
                dV[b, lo:p + 1, g] += np.outer(P_w, dO[b, t, h])
    assert np.allclose(o, ref["o"], rtol=1e-10, atol=1e-12)
    for got, want, name in ((dQ, dQ_ref, "dQ"), (dK, dK_ref, "dK"), (dV, dV_ref, "dV")):
        assert np.allclose(got, want, rtol=1e-9, atol=1e-11), name
