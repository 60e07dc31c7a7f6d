"""GPU parity of the backward (dQ, dK, dV, dgate) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import Case, check_close, check_backward_full, check_same_or_rounding, run_backward, to_f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,Lq,Lk,Hq,Hkv,D,W,rho", [
    (1, 1024, 1024, 1, 1, 64, 128, 0.2),     # the tiny configuration's shape, with a backward
    (1, 700, 700, 2, 1, 128, 200, 0.3),      # ragged tail, window not a block multiple
    (2, 513, 513, 4, 2, 128, 128, 0.5),      # batch > 1, GQA group sums
    (1, 300, 1000, 2, 2, 64, 96, 0.4),       # Lk > Lq: keys nobody sees get zero gradients
    (1, 640, 640, 2, 1, 128, 0, 0.2),        # W = 0
    (1, 600, 600, 1, 1, 64, 5000, 0.2),      # W >= L - 1
    (1, 1, 1, 1, 1, 128, 4, 1.0),            # single token
    (1, 129, 129, 1, 1, 128, 16, 1.0),       # all routed
    (1, 1500, 1500, 2, 2, 128, 256, 0.02),   # few routed rows
    (1, 900, 900, 2, 1, 128, 300, 0.0),      # nothing routed: pure sliding-window backward
])
def test_backward_matches_oracle(B, Lq, Lk, Hq, Hkv, D, W, rho):
    d = synth.mask_bernoulli(B, Lq, rho, seed=Lq * 3 + W)
    c = Case(B, Lq, Hq, Hkv, D, W, d, seed=Lq + 17 * D + W, Lk=Lk, backward=True)
    c.run_forward()
    c.check_forward_full()
    run_backward(c)
    check_backward_full(c)
    # dgate: sum over heads of dO_t . a_t on routed rows (first term of Eq. 7), zero elsewhere
    ref = c.oracle_forward()
    want = (ref["a"] * to_f64(c.buf.dO)).sum(axis=(2, 3)) * d
    check_close(to_f64(c.buf.dgate), want, "dgate", 5e-2, 5e-3)


def test_backward_identities_at_length():
    """O(L) identities that hold at any size: sum_j dV_j = sum_t (1 + d_t) dO_t per KV group; V == const -> dQ = dK = 0."""
    B, L, Hq, Hkv, D, W = 1, 6000, 4, 2, 128, 1024
    d = synth.mask_clustered(B, L, 0.3, seed=8)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=99, backward=True)
    c.run_forward()
    run_backward(c)
    dO = to_f64(c.buf.dO)
    want = (dO * (1 + d)[:, :, None, None]).reshape(B, L, Hkv, Hq // Hkv, D).sum(axis=(1, 3))
    got = to_f64(c.buf.dV).sum(axis=1)
    assert np.abs(got - want).max() <= 0.5, np.abs(got - want).max()     # sums of 6000 bf16-rounded rows
    c.buf.V.copy_(torch.ones_like(c.buf.V) * 0.5)
    c.run_forward()
    run_backward(c)
    assert to_f64(c.buf.dQ).__abs__().max() <= 2e-2
    assert to_f64(c.buf.dK).__abs__().max() <= 2e-2


def test_backward_run_twice():
    """dK and dV are summed on chip in a fixed order: bit-identical from run to run.  dQ is summed over the key blocks with
    atomic fp32 additions in no fixed order: equal up to the rounding of sums that differ in their last bits."""
    B, L, Hq, Hkv, D, W = 1, 777, 2, 1, 128, 100
    d = synth.mask_bernoulli(B, L, 0.3, seed=2)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=3, backward=True)
    c.run_forward()
    run_backward(c)
    first = [t.clone() for t in (c.buf.dQ, c.buf.dK, c.buf.dV)]
    run_backward(c)
    check_same_or_rounding(first[0], c.buf.dQ, "dQ")
    for x, y in zip(first[1:], (c.buf.dK, c.buf.dV)):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))
