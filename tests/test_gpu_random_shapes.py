"""Seeded random problem shapes: forward and backward parity against the fp64 oracle on shapes nobody picked by
hand (ragged lengths, more keys than queries, every group size up to 8, both head sizes, windows from 0 to beyond
the sequence, routed densities from none to all)."""
import numpy as np
import pytest

from paper_2603_17484_b200 import synth
from tests.gpu_util import Case, check_backward_full, run_backward

pytestmark = pytest.mark.gpu


def _shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        B = int(rng.integers(1, 4))
        Lq = int(rng.choice([1, 2, 63, 127, 128, 129, 255, 257, 300, 511, 640, 777]))
        Lk = Lq + int(rng.choice([0, 0, 0, 1, 37, 128, 300]))
        Hkv = int(rng.integers(1, 3))
        G = int(rng.choice([1, 2, 3, 4, 7, 8]))
        D = int(rng.choice([64, 128]))
        W = int(rng.choice([0, 1, 17, 127, 128, 200, 512, 4096]))
        rho = float(rng.choice([0.0, 0.05, 0.3, 0.7, 1.0]))
        out.append((B, Lq, Lk, Hkv * G, Hkv, D, W, rho, 1000 + i))
    return out


@pytest.mark.parametrize("B,Lq,Lk,Hq,Hkv,D,W,rho,seed", _shapes(24, 20260317))
def test_random_shape(B, Lq, Lk, Hq, Hkv, D, W, rho, seed):
    d = synth.mask_bernoulli(B, Lq, rho, seed=seed)
    c = Case(B, Lq, Hq, Hkv, D, W, d, seed=seed + 1, Lk=Lk, backward=True)
    c.run_forward()
    c.check_forward_full()
    run_backward(c)
    check_backward_full(c)
