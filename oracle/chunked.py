"""Running (online) soft-max attention over an arbitrary partition of the keys, numpy fp64.  TEST INFRASTRUCTURE ONLY.

The CUDA kernels never see a whole score row: they visit the keys in chunks, carry (maximum, sum, weighted values)
from chunk to chunk, and stop at the chunk that holds the last visible key of a group of rows -- the evaluation order
of Algorithm 1.  This module states that order for ANY chunk boundaries and ANY grouping of rows, so the tests can
require it to equal the plain two-pass definition in ``l2a_oracle.c`` (to 1e-12) for uniform, ragged and random
chunkings alike.

Readings of Algorithm 1 that the equality depends on (0-based positions): a group of rows visits the chunks up to and
including the one that holds its largest position; the carried values and the carried sum are rescaled by the same
factor when the maximum moves; the log-sum-exp is formed from the statistics after the last visited chunk.
"""
from __future__ import annotations

import numpy as np


def merge_chunk(state, scores, values):
    """One step of the running soft-max.  state = (m [r], l [r], acc [r, d]); scores [r, c] with -inf for masked pairs;
    values [c, d].  Returns the state after the chunk."""
    m, l, acc = state
    m_next = np.maximum(m, scores.max(axis=1, initial=-np.inf))
    ref = np.where(np.isfinite(m_next), m_next, 0.0)          # a row that has seen no key yet keeps a zero state
    keep = np.where(np.isfinite(m), np.exp(m - ref), 0.0)
    p = np.exp(scores - ref[:, None])
    return m_next, keep * l + p.sum(axis=1), keep[:, None] * acc + p @ values


def attend_chunked(q, K, V, pos, bounds, scale=None, lowest=None):
    """Rows ``q`` [r, d] at key positions ``pos`` [r] attend causally (key <= pos, and key >= lowest if given) over
    the key chunks ``bounds`` = [0 = b_0 < b_1 < ... < b_m = n]; chunks wholly after the group's largest position are
    not visited.  Returns (out [r, d], lse [r], chunks visited)."""
    q, K, V = (np.asarray(x, np.float64) for x in (q, K, V))
    pos = np.asarray(pos, np.int64)
    scale = 1.0 / np.sqrt(K.shape[1]) if scale is None else scale
    r = q.shape[0]
    state = (np.full(r, -np.inf), np.zeros(r), np.zeros((r, V.shape[1])))
    visited = 0
    for lo, hi in zip(bounds[:-1], bounds[1:]):
        if lo > pos.max():
            break
        keys = np.arange(lo, hi)
        ok = keys[None, :] <= pos[:, None]
        if lowest is not None:
            ok &= keys[None, :] >= np.asarray(lowest)[:, None]
        state = merge_chunk(state, np.where(ok, (q @ K[lo:hi].T) * scale, -np.inf), V[lo:hi])
        visited += 1
    m, l, acc = state
    return acc / l[:, None], m + np.log(l), visited
