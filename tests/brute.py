"""Brute-force pins for the oracle: explicit L x L mask matrices, row soft-max, matmul (numpy fp64).

Written directly from the mask definitions of Section 2 (causal: j <= i; sliding window:
0 <= i - j <= w) and Eq. 2-5; deliberately shares nothing with ``oracle/``."""
import numpy as np


def bf16_bits_to_f64(u16: np.ndarray) -> np.ndarray:
    return (u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit patterns (inputs assumed finite)."""
    u = np.asarray(x, np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + r) >> 16).astype(np.uint16)


def masked_attention(q, k, v, mask_add, scale):
    """q [Lq, D], k/v [Lk, D], mask_add [Lq, Lk] of 0 / -inf."""
    s = (q @ k.T) * scale + mask_add
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=1, keepdims=True)
    return (e / l) @ v, (m + np.log(l))[:, 0]


def layer_brute(Q, K, V, d, W, scale=None, offset=None):
    """Q [B, Lq, Hq, D], K/V [B, Lk, Hkv, D] fp64; d [B, Lq] 0/1.  Returns dict like the oracle."""
    B, Lq, Hq, D = Q.shape
    Lk, Hkv = K.shape[1], K.shape[2]
    G = Hq // Hkv
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    offset = Lk - Lq if offset is None else offset
    i = np.arange(Lq)[:, None] + offset
    j = np.arange(Lk)[None, :]
    M_causal = np.where(j <= i, 0.0, -np.inf)
    M_window = np.where((i - j >= 0) & (i - j <= W), 0.0, -np.inf)
    s = np.zeros_like(Q)
    a = np.zeros_like(Q)
    lse_loc = np.zeros((B, Hq, Lq))
    lse_glb = np.full((B, Hq, Lq), np.nan)
    for b in range(B):
        for h in range(Hq):
            g = h // G
            s[b, :, h], lse_loc[b, h] = masked_attention(Q[b, :, h], K[b, :, g], V[b, :, g], M_window, scale)
            ag, lg = masked_attention(Q[b, :, h], K[b, :, g], V[b, :, g], M_causal, scale)
            on = d[b].astype(bool)
            a[b, on, h] = ag[on]
            lse_glb[b, h, on] = lg[on]
    return {"s": s, "a": a, "o": s + a, "lse_loc": lse_loc, "lse_glb": lse_glb}
