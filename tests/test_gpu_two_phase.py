"""The layer in the order the paper defines it (Eq. 2 -> 3 -> 4 -> 5): local attention, router logits from the local
output, routing + compaction, then global attention for the routed tokens added into the output.  The two-phase
result must equal the single-call result for the same routing mask, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import Case, check_close, check_backward_full, run_backward, to_f64

pytestmark = pytest.mark.gpu


def test_two_phase_layer_matches_single_call():
    B, L, Hq, Hkv, D, W = 2, 1100, 4, 2, 128, 192
    c = Case(B, L, Hq, Hkv, D, W, np.zeros((B, L), np.uint8), seed=71, backward=True)
    b = c.buf
    # phase 1: local attention only
    p1 = l2a.params(B, L, L, Hq, Hkv, D, W, flags=l2a.FLAG_SAVE_FOR_BWD | l2a.FLAG_SKIP_GLOBAL)
    l2a.l2a_forward(p1, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.O, b.S_save, b.A_c, b.lse_loc,
                    b.lse_glb, b.fwd_ws)
    # router on the local output (Eq. 3); weights chosen so that roughly a quarter of the tokens are routed
    rng = np.random.default_rng(3)
    w = torch.from_numpy((rng.standard_normal(Hq * D) * 0.5).astype(np.float32)).cuda()
    logits = torch.empty((B, L), dtype=torch.float32, device="cuda")
    sum_sq = torch.empty((B,), dtype=torch.float32, device="cuda")
    l2a.l2a_router_logits(p1, b.S_save, w, -0.3, logits, sum_sq)
    torch.cuda.synchronize()
    S_bits = b.S_save.cpu().view(torch.int16).numpy().view(np.uint16)
    z_ref = oracle.router_logits(S_bits, w.cpu().numpy(), -0.3)
    z = logits.cpu().numpy()
    assert np.abs(z - z_ref).max() <= 1e-3 * (1 + np.abs(z_ref).max())
    # the regulariser's sum (Eq. 6) of the kernel's own fp32 logits: fp32 sigmoid and an atomic fp32 sum
    want_sq = oracle.gate_regulariser_sum(z.astype(np.float64))
    assert np.abs(sum_sq.cpu().numpy().astype(np.float64) - want_sq).max() <= 1e-4 * want_sq.max()
    # the decision is taken on the kernel's own fp32 logits: integer results are then exact
    d = oracle.route(z, 0.0)
    assert 0.02 < d.mean() < 0.9
    l2a.l2a_route_compact(p1, logits, l2a.ROUTER_LOGITS_F32, 0.0, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.route_ws)
    # phase 2: global attention of the routed tokens, added into O
    p2 = l2a.params(B, L, L, Hq, Hkv, D, W, flags=l2a.FLAG_SAVE_FOR_BWD | l2a.FLAG_GLOBAL_PHASE)
    l2a.l2a_forward(p2, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.O, b.S_save, b.A_c, b.lse_loc,
                    b.lse_glb, b.fwd_ws)
    torch.cuda.synchronize()
    assert np.array_equal(b.d_mask.cpu().numpy(), d)
    two_phase = {k: getattr(b, k).clone() for k in ("O", "S_save", "lse_loc")}
    n = b.n_routed.cpu().numpy()
    A_two = b.A_c.clone()
    # single call with the same mask
    c.d = d
    b.router = torch.from_numpy(d).cuda()
    c.kind = l2a.ROUTER_MASK_U8
    c.run_forward()
    ref = c.check_forward_full()
    for k, v in two_phase.items():
        assert torch.equal(v.view(torch.int16) if v.dtype == torch.bfloat16 else v, getattr(b, k).view(torch.int16) if v.dtype == torch.bfloat16 else getattr(b, k)), k
    for bi in range(B):
        assert torch.equal(A_two[bi, :n[bi]].view(torch.int16), b.A_c[bi, :n[bi]].view(torch.int16))
    run_backward(c)
    check_backward_full(c)
