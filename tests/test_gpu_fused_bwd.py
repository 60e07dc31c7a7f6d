"""L2A_FLAG_FUSED_DQ: the backward with dQ produced inside the dK/dV kernel (five GEMMs per tile pair) and summed in
fp32 accumulators.  Same parity bar against the fp64 oracle as the seven-GEMM path."""
import numpy as np
import pytest
import torch

from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import MAX_ABS, Case, check_backward_full, check_close, run_backward, to_f64

pytestmark = pytest.mark.gpu


def fused_backward(c, extra_flags=0):
    b, s = c.buf, c.shape
    p = l2a.params(s.B, s.Lq, s.Lk, s.Hq, s.Hkv, s.D, s.window,
                   flags=l2a.FLAG_SAVE_FOR_BWD | l2a.FLAG_FUSED_DQ | extra_flags)
    ws = torch.empty(l2a.l2a_workspace_bytes(p)[2], dtype=torch.uint8, device="cuda")
    for t in (b.dQ, b.dK, b.dV):
        t.fill_(float("nan"))
    l2a.l2a_backward(p, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.dO, b.S_save, b.A_c, b.lse_loc,
                     b.lse_glb, b.dQ, b.dK, b.dV, b.dgate, ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(ws) == 0


@pytest.mark.parametrize("B,Lq,Lk,Hq,Hkv,D,W,rho", [
    (1, 700, 700, 2, 1, 128, 200, 0.3),
    (2, 513, 513, 4, 2, 128, 128, 0.5),
    (1, 300, 1000, 2, 2, 64, 96, 0.4),
    (1, 1500, 1500, 8, 2, 128, 256, 0.1),
    (1, 129, 129, 1, 1, 128, 16, 1.0),
    (1, 900, 900, 2, 1, 64, 300, 0.0),
    (1, 1, 1, 1, 1, 128, 4, 1.0),
])
@pytest.mark.parametrize("shared", [False, True], ids=["plain", "shared_window"])
def test_fused_backward_matches_oracle(B, Lq, Lk, Hq, Hkv, D, W, rho, shared):
    d = synth.mask_bernoulli(B, Lq, rho, seed=Lq + W)
    c = Case(B, Lq, Hq, Hkv, D, W, d, seed=Lq + 3 * D, Lk=Lk, backward=True)
    c.run_forward()
    run_backward(c)
    plain = {k: getattr(c.buf, k).clone() for k in ("dQ", "dK", "dV")}
    fused_backward(c, l2a.FLAG_SHARED_WINDOW if shared else 0)
    b = c.buf
    check_backward_full(c, dq_first_rows=4)
    check_close(to_f64(b.dQ), to_f64(plain["dQ"]), "dQ fused vs seven-GEMM path", max_abs=2 * MAX_ABS)
    check_close(to_f64(b.dK), to_f64(plain["dK"]), "dK fused vs seven-GEMM path", max_abs=2 * MAX_ABS)
    check_close(to_f64(b.dV), to_f64(plain["dV"]), "dV fused vs seven-GEMM path", max_abs=2 * MAX_ABS)
