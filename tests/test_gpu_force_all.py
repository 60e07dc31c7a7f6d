"""Training-mode pass that runs Global Attention for every token (Section 3.3, footnote): the output and the
attention gradients are unchanged, the global output is available for every token, and the loss term of the
straight-through router gradient (Eq. 7), dgate_t = sum_h dO_t . a_t, covers every token."""
import numpy as np
import pytest

import oracle
from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import Case, check_close, check_backward_full, run_backward, to_f64, LSE_ABS

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,L,Hq,Hkv,D,W,rho", [
    (1, 700, 2, 1, 128, 200, 0.3),
    (2, 513, 4, 2, 128, 64, 0.1),
    (1, 640, 2, 2, 64, 96, 0.5),
    (1, 300, 1, 1, 128, 32, 0.0),      # nothing routed: O = S, yet every token gets a gate gradient
])
def test_force_all_global_forward_backward(B, L, Hq, Hkv, D, W, rho):
    d = synth.mask_bernoulli(B, L, rho, seed=L + W)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=5 * L + D, backward=True, flags=l2a.FLAG_FORCE_ALL_GLOBAL)
    c.run_forward()
    c.check_routing()
    ref = c.oracle_forward()                                            # with the real routing mask
    ones = np.ones_like(d)
    ref_all = oracle.forward_full(c.shape, c.u16("Q"), c.u16("K"), c.u16("V"), ones)   # a_t for every token
    check_close(to_f64(c.buf.O), ref["o"], "O (forced pass leaves the output unchanged)")
    check_close(to_f64(c.buf.S_save), ref["s"], "S_save")
    check_close(to_f64(c.buf.A_c), ref_all["a"], "A by row")
    check_close(to_f64(c.buf.lse_glb), ref_all["lse_glb"], "lse_glb by row", LSE_ABS, LSE_ABS)
    run_backward(c)
    check_backward_full(c)                                              # same dQ, dK, dV as the conditional pass
    rb, rt = np.meshgrid(np.arange(B), np.arange(L), indexing="ij")
    want = oracle.dgate_rows(c.shape, c.u16("Q"), c.u16("K"), c.u16("V"), c.u16("dO"), rb.ravel(), rt.ravel())
    check_close(to_f64(c.buf.dgate), want.reshape(B, L), "dgate (every token)", 5e-2, 5e-3)


def test_force_all_requires_saving():
    p = l2a.params(1, 256, 256, 2, 1, 128, 16, flags=l2a.FLAG_FORCE_ALL_GLOBAL)   # without SAVE_FOR_BWD
    buf = l2a.Buffers.allocate(p)
    assert l2a.l2a_forward(p, buf.Q, buf.K, buf.V, buf.d_mask, buf.q_idx, buf.n_routed, buf.prefix, buf.O, None, None,
                           None, None, buf.fwd_ws, check=False) == -1
