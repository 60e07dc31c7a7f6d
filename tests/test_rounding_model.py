"""Where the gradient tolerance of the GPU parity tests comes from (CPU only).

The kernels keep scores, soft-max and accumulators in fp32 but feed the tensor cores bf16 operands: P is rounded to
bf16 before dV = P^T dO, dS = P (dP - Delta) is formed from that rounded P and rounded to bf16 before dK = dS^T Q and
dQ = dS K, Delta uses the stored bf16 outputs, and every result is rounded to bf16 once.  This test applies exactly
those roundings to a plain fp64 evaluation of the backward (numpy, written from the definition; nothing shared with
the CUDA path or the C oracle) on shapes of tests/test_gpu_backward.py and compares with the oracle:

  * without the roundings the evaluation equals the oracle to 1e-12 (so the model is the same function);
  * with them, some elements leave the plain bound 2e-2 (large dK / dV entries cannot even be stored that accurately),
    which is why the bound carries the 2^-8 |want| term;
  * against 2e-2 + 2^-8 |want|, rows and keys beyond the first eight have rare, small excursions (at most one element per
    array, never beyond 1.1 x the bound; tests/gpu_util.py allows a 1e-5 fraction up to 1.5 x);
  * the first eight rows / keys, which see a handful of keys / are seen through rows with a handful of keys, can exceed
    the bound in a few elements per head (the error of Delta is not averaged out there), by at most 1.7 x here;
    tests/gpu_util.py allows 8 elements per (batch, head) up to 2 x.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2603_17484_b200 import synth


def bf16_round(x):
    """nearest bf16 (ties to even) of an fp64 / fp32 array, as fp64"""
    f = np.asarray(x, np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return r.astype(np.uint32).view(np.float32).astype(np.float64)


def from_bits(a):
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def backward_model(B, Lq, Lk, Hq, Hkv, D, W, d, t, rounded):
    Q, K, V, dO = (from_bits(synth.as_u16(t[k])) for k in ("Q", "K", "V", "dO"))
    scale = 1.0 / math.sqrt(D)
    G, off = Hq // Hkv, Lk - Lq
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)
    rnd = bf16_round if rounded else (lambda x: x)
    for b in range(B):
        pos = np.arange(Lq)[:, None] + off
        key = np.arange(Lk)[None, :]
        masks = ((key <= pos) & (key >= pos - W), (key <= pos) & (d[b][:, None] != 0))
        for h in range(Hq):
            g = h // G
            q, k, v, do = Q[b, :, h], K[b, :, g], V[b, :, g], dO[b, :, h]
            s = scale * (q @ k.T)
            for m in masks:
                rows = m.any(axis=1, keepdims=True)
                if not rows.any():
                    continue
                sm = np.where(m, s, -np.inf)
                mx = np.max(sm, axis=1, keepdims=True)
                mx[~np.isfinite(mx)] = 0.0
                e = np.where(m, np.exp(sm - mx), 0.0)
                l = e.sum(axis=1, keepdims=True)
                l[l == 0] = 1.0
                p = e / l
                # the forward's output: probabilities rounded to bf16 before P V, normalised by the fp32 row sum,
                # stored as bf16; Delta is formed from that stored output
                delta = (do * rnd((rnd(e) @ v) / l)).sum(axis=1, keepdims=True)
                pb = rnd(p)
                ds = rnd(pb * (do @ v.T - delta)) * rows
                dV[b, :, g] += pb.T @ (do * rows)
                dK[b, :, g] += scale * (ds.T @ q)
                dQ[b, :, h] += scale * (ds @ k)
    return rnd(dQ), rnd(dK), rnd(dV)


EARLY = 8     # the first rows / keys, treated separately (tests/gpu_util.EARLY_ROWS)

CASES = [
    (1, 1024, 1024, 1, 1, 64, 128, 0.2),
    (1, 700, 700, 2, 1, 128, 200, 0.3),
    (2, 513, 513, 4, 2, 128, 128, 0.5),
    (1, 129, 129, 1, 1, 128, 16, 1.0),
]


@pytest.mark.parametrize("B,Lq,Lk,Hq,Hkv,D,W,rho", CASES)
def test_operand_roundings_explain_the_gradient_tolerance(B, Lq, Lk, Hq, Hkv, D, W, rho):
    d = synth.mask_bernoulli(B, Lq, rho, seed=Lq * 3 + W)
    t = synth.qkv(B, Lq, Hq, Hkv, D, Lq + 17 * D + W, with_dO=True, Lk=Lk)
    sh = oracle.Shape(B, Lq, Lk, Hq, Hkv, D, W)
    want = oracle.backward_full(sh, *(synth.as_u16(t[k]) for k in ("Q", "K", "V")), d, synth.as_u16(t["dO"]))
    exact = backward_model(B, Lq, Lk, Hq, Hkv, D, W, d, t, rounded=False)
    for g, w in zip(exact, want):
        assert np.abs(g - w).max() <= 1e-12 * max(1.0, np.abs(w).max())
    got = backward_model(B, Lq, Lk, Hq, Hkv, D, W, d, t, rounded=True)
    over_plain = 0
    for name, g, w in zip(("dQ", "dK", "dV"), got, want):
        err = np.abs(g - w)
        bound = 2e-2 + 2.0 ** -8 * np.abs(w)
        over_plain += int((err > 2e-2).sum())
        late, late_b = err[:, EARLY:], bound[:, EARLY:]
        if late.size:
            assert int((late > late_b).sum()) <= 1, name                  # the GPU tests allow ceil(1e-5 * size) >= 1
            assert (late / late_b).max() <= 1.1, (name, (late / late_b).max())  # the GPU tests allow 1.5
        early = (err[:, :EARLY] > bound[:, :EARLY]).sum(axis=(1, 3))
        assert early.max() <= 6, (name, early)                            # the GPU tests allow 8 per (batch, head)
        assert (err[:, :EARLY] / bound[:, :EARLY]).max() <= 1.7, name     # the GPU tests allow 2
        assert err.mean() <= 0.5 * (2e-3 + 2.0 ** -9 * np.abs(w).mean()), (name, err.mean())
    if (B, Lq) == (2, 513):
        # large dK / dV entries of early keys (sums over ~2000 rows) cannot be stored in bf16 to within 2e-2
        assert over_plain > 0


def test_first_rows_exceed_the_bound_only_slightly():
    """All tokens routed, four query heads per KV head: the configuration in which the error of Delta adds up most (both
    modules see the same few keys; dK sums the heads).  Over 40 seeds the excursions stay within the first rows / keys,
    at most five elements per head, at most 1.7 x the bound -- and they do occur, so the looser rule is needed."""
    B, Lq, Lk, Hq, Hkv, D, W = 1, 64, 64, 4, 1, 128, 16
    seen = 0
    for sd in range(40):
        d = np.ones((B, Lq), np.uint8)
        t = synth.qkv(B, Lq, Hq, Hkv, D, 5000 + sd, with_dO=True, Lk=Lk)
        sh = oracle.Shape(B, Lq, Lk, Hq, Hkv, D, W)
        want = oracle.backward_full(sh, *(synth.as_u16(t[k]) for k in ("Q", "K", "V")), d, synth.as_u16(t["dO"]))
        got = backward_model(B, Lq, Lk, Hq, Hkv, D, W, d, t, rounded=True)
        for g, w in zip(got, want):
            err = np.abs(g - w)
            bound = 2e-2 + 2.0 ** -8 * np.abs(w)
            over = err > bound
            seen += int(over.sum())
            assert not over[:, EARLY:].any()
            assert over[:, :EARLY].sum(axis=(1, 3)).max() <= 6
            assert (err / bound).max() <= 1.7
    assert seen > 0
