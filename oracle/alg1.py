"""Algorithm 1 (L2A kernel forward pass) restated in numpy fp64.  TEST INFRASTRUCTURE ONLY.

Single sequence, single head: compacted routed queries are tiled, each tile walks the key/value
tiles up to its own causal bound with an online soft-max, and the compact result is scattered back.
It exists to check that the algorithm's steps, read with the corrections below, give the plain
definition in ``l2a_oracle.c``; the tests require the two to agree to 1e-12.

Readings of the printed algorithm taken here (0-based positions):
  * the index list has length n_c (routed count) and is tiled into ceil(n_c / B_q) blocks;
  * the per-tile key-block bound is ceil((max(Q_idx tile) + 1) / B_k);
  * the running output is rescaled by the SAME factor exp(m_old - m_new) as the running sum
    (no inverse), otherwise the final division by the running sum would not normalise;
  * the finalisation uses the statistics after the last visited key tile;
  * a ragged last tile is padded with masked rows that are never written back.
"""
from __future__ import annotations

import numpy as np


def l2a_alg1_forward(Q, K, V, q_idx, Bq: int, Bk: int, scale: float | None = None):
    """Q, K, V fp64 [n, d]; q_idx ascending int positions of routed queries.

    Returns (O [n, d] zero outside q_idx, O_c [n_c, d], L_c [n_c])."""
    Q = np.asarray(Q, np.float64)
    K = np.asarray(K, np.float64)
    V = np.asarray(V, np.float64)
    q_idx = np.asarray(q_idx, np.int64)
    n, d = K.shape
    n_c = q_idx.size
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    Q_c = Q[q_idx]                                   # step 1: consolidate active queries
    T_q = -(-n_c // Bq)
    O = np.zeros((Q.shape[0], d))                    # step 3: zero-initialised full output
    O_c = np.zeros((n_c, d))
    L_c = np.zeros((n_c,))
    for i in range(T_q):
        rows = slice(i * Bq, min((i + 1) * Bq, n_c))
        Qi = Q_c[rows]
        idx_i = q_idx[rows]
        max_k_blocks = -(-(int(idx_i.max()) + 1) // Bk)
        Oi = np.zeros((Qi.shape[0], d))
        li = np.zeros((Qi.shape[0],))
        mi = np.full((Qi.shape[0],), -np.inf)
        for j in range(max_k_blocks):
            k_idx = np.arange(j * Bk, min((j + 1) * Bk, n))
            Kj, Vj = K[k_idx], V[k_idx]
            S = (Qi @ Kj.T) * scale
            S = np.where(idx_i[:, None] >= k_idx[None, :], S, -np.inf)
            m_new = np.maximum(mi, S.max(axis=1))
            m_safe = np.where(np.isfinite(m_new), m_new, 0.0)   # rows with no visible key yet
            P = np.exp(S - m_safe[:, None])
            alpha = np.where(np.isfinite(mi), np.exp(mi - m_safe), 0.0)
            li = alpha * li + P.sum(axis=1)
            Oi = alpha[:, None] * Oi + P @ Vj
            mi = m_new
        O_c[rows] = Oi / li[:, None]
        L_c[rows] = mi + np.log(li)
    O[q_idx] = O_c                                   # scatter
    return O, O_c, L_c
