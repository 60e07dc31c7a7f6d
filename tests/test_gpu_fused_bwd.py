"""L2A_FLAG_FUSED_DQ: the backward with dQ produced inside the dK/dV kernel (five GEMMs per tile pair) and summed in an
fp32 buffer.  Same parity bar against the fp64 oracle; dK and dV equal the seven-GEMM path bit for bit (same
arithmetic), dQ only within rounding (the fp32 sums are taken in a different order)."""
import numpy as np
import pytest
import torch

from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import MAX_ABS, Case, check_backward_full, check_close, run_backward, to_f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,Lq,Lk,Hq,Hkv,D,W,rho", [
    (1, 700, 700, 2, 1, 128, 200, 0.3),
    (2, 513, 513, 4, 2, 128, 128, 0.5),
    (1, 300, 1000, 2, 2, 64, 96, 0.4),
    (1, 1500, 1500, 8, 2, 128, 256, 0.1),
    (1, 129, 129, 1, 1, 128, 16, 1.0),
    (1, 900, 900, 2, 1, 64, 300, 0.0),
    (1, 1, 1, 1, 1, 128, 4, 1.0),
])
def test_fused_backward_matches_oracle(B, Lq, Lk, Hq, Hkv, D, W, rho):
    d = synth.mask_bernoulli(B, Lq, rho, seed=Lq + W)
    c = Case(B, Lq, Hq, Hkv, D, W, d, seed=Lq + 3 * D, Lk=Lk, backward=True)
    c.run_forward()
    run_backward(c)
    plain = {k: getattr(c.buf, k).clone() for k in ("dQ", "dK", "dV")}
    b = c.buf
    p = l2a.params(B, Lq, Lk, Hq, Hkv, D, W, flags=l2a.FLAG_SAVE_FOR_BWD | l2a.FLAG_FUSED_DQ)
    ws = torch.empty(l2a.l2a_workspace_bytes(p)[2], dtype=torch.uint8, device="cuda")
    for t in (b.dQ, b.dK, b.dV):
        t.fill_(float("nan"))
    l2a.l2a_backward(p, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.dO, b.S_save, b.A_c, b.lse_loc,
                     b.lse_glb, b.dQ, b.dK, b.dV, b.dgate, ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(ws) == 0
    check_backward_full(c, dq_first_rows=4)
    assert torch.equal(b.dK.view(torch.int16), plain["dK"].view(torch.int16))
    assert torch.equal(b.dV.view(torch.int16), plain["dV"].view(torch.int16))
    # the two dQ are bf16 results with independent errors against the exact value (order of the fp32 additions, P
    # rounded to bf16 or not inside dS, one more bf16 rounding where the seven-GEMM path adds the global part to the
    # rounded local part): against each other they get twice the bound each one has against the oracle
    check_close(to_f64(b.dQ), to_f64(plain["dQ"]), "dQ fused vs seven-GEMM path", max_abs=2 * MAX_ABS)


def test_fused_rejects_partial_backward_flags():
    """The fused kernel always runs both attention sets: the partial-backward and forced-global flags are refused."""
    d = synth.mask_bernoulli(1, 200, 0.5, seed=5)
    c = Case(1, 200, 2, 1, 128, 64, d, seed=9, backward=True)
    c.run_forward()
    b = c.buf
    for extra in (l2a.FLAG_SKIP_LOCAL, l2a.FLAG_SKIP_GLOBAL, l2a.FLAG_FORCE_ALL_GLOBAL):
        p = l2a.params(1, 200, 200, 2, 1, 128, 64, flags=l2a.FLAG_SAVE_FOR_BWD | l2a.FLAG_FUSED_DQ | extra)
        ws = torch.empty(l2a.l2a_workspace_bytes(p)[2], dtype=torch.uint8, device="cuda")
        with pytest.raises(l2a.L2AError):
            l2a.l2a_backward(p, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.dO, b.S_save, b.A_c,
                             b.lse_loc, b.lse_glb, b.dQ, b.dK, b.dV, b.dgate, ws)
