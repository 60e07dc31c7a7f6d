"""Host-side arithmetic of bench.py that the reported figures rest on (no GPU)."""
import numpy as np

import bench
from paper_2603_17484_b200 import synth


def brute_tile_pairs(mask_row, L, W, T, shared):
    """(tile, block) pairs that hold at least one visible (query, key) pair, by enumeration; the launches issue the
    contiguous range from the first to the last such block of a tile."""
    loc = 0
    for r0 in range(0, L, T):
        rows = np.arange(r0, min(r0 + T, L))
        blocks = set()
        for t in rows:
            blocks.update(range(max(t - W, 0) // T, t // T + 1))
        loc += max(blocks) - min(blocks) + 1
    glb = 0
    routed = np.nonzero(mask_row)[0]
    for c0 in range(0, len(routed), T):
        rows = routed[c0:c0 + T]
        hi = [t - (W + 1 if shared else 0) for t in rows]
        hi = [h for h in hi if h >= 0]
        if hi:
            glb += max(hi) // T + 1                       # blocks 0 .. the one holding the last visible key
    return loc * T * T, glb * T * T


def test_issued_tile_pairs_match_enumeration():
    rng = np.random.default_rng(3)
    for L, W, T, rho in [(1000, 100, 128, 0.3), (517, 0, 128, 0.5), (2048, 4096, 128, 0.1), (300, 64, 32, 1.0), (900, 200, 128, 0.0)]:
        mask = (rng.random((2, L)) < rho).astype(np.uint8)
        for shared in (False, True):
            got = bench.issued_tile_pairs(mask, L, W, shared, tile=T)
            want = [sum(x) for x in zip(*(brute_tile_pairs(mask[b], L, W, T, shared) for b in range(2)))]
            assert list(got) == want, (L, W, T, rho, shared)


def test_issued_pairs_cover_the_useful_ones():
    L, W = 4096, 512
    mask = synth.mask_clustered(1, L, 0.2, 11)
    loc, glb = bench.issued_tile_pairs(mask, L, W)
    assert loc >= synth.pairs_local(L, W) and glb >= synth.pairs_global(mask[0])
    assert loc < 1.3 * synth.pairs_local(L, W)
