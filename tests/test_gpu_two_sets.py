"""A layer whose Global Attention has its own Q/K/V (its own projections of the local output, Section 3.1): the
forward is the local phase on one set and the global phase on the other; the backward is one call per module."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import Case, check_close, check_same_or_rounding, to_f64

pytestmark = pytest.mark.gpu


def test_separate_qkv_for_the_global_module():
    B, L, Hq, Hkv, D, W = 2, 1000, 4, 2, 128, 150
    d = synth.mask_bernoulli(B, L, 0.25, seed=12)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=61, backward=True)          # local set + dO
    b = c.buf
    g = synth.qkv(B, L, Hq, Hkv, D, seed=62)                          # global set
    Qg, Kg, Vg = (g[k].cuda() for k in ("Q", "K", "V"))
    b.route(c.kind, c.threshold)
    flags = l2a.FLAG_SAVE_FOR_BWD
    p_loc = l2a.params(B, L, L, Hq, Hkv, D, W, flags=flags | l2a.FLAG_SKIP_GLOBAL)
    p_glb = l2a.params(B, L, L, Hq, Hkv, D, W, flags=flags | l2a.FLAG_GLOBAL_PHASE)
    b.O.fill_(float("nan"))
    l2a.l2a_forward(p_loc, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.O, b.S_save, b.A_c, b.lse_loc,
                    b.lse_glb, b.fwd_ws)
    l2a.l2a_forward(p_glb, Qg, Kg, Vg, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.O, b.S_save, b.A_c, b.lse_loc,
                    b.lse_glb, b.fwd_ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(b.fwd_ws) == 0
    ref_loc = oracle.forward_full(c.shape, c.u16("Q"), c.u16("K"), c.u16("V"), np.zeros_like(d))
    gu = {k: synth.as_u16(g[k]) for k in ("Q", "K", "V")}
    ref_glb = oracle.forward_full(c.shape, gu["Q"], gu["K"], gu["V"], d)
    want = ref_loc["s"] + d[:, :, None, None] * ref_glb["a"]                   # Eq. 5 with a_t from the global set
    check_close(to_f64(b.O), want, "O with two Q/K/V sets")

    # backward: one call per module
    dQ, dK, dV = b.dQ, b.dK, b.dV
    dQg, dKg, dVg = torch.empty_like(dQ), torch.empty_like(dK), torch.empty_like(dV)
    for t in (dQ, dK, dV, dQg, dKg, dVg):
        t.fill_(float("nan"))
    pb_loc = l2a.params(B, L, L, Hq, Hkv, D, W, flags=flags | l2a.FLAG_SKIP_GLOBAL)
    pb_glb = l2a.params(B, L, L, Hq, Hkv, D, W, flags=flags | l2a.FLAG_SKIP_LOCAL)
    l2a.l2a_backward(pb_loc, b.Q, b.K, b.V, None, None, None, None, b.dO, b.S_save, None, b.lse_loc, None, dQ, dK, dV,
                     None, b.bwd_ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(b.bwd_ws) == 0
    l2a.l2a_backward(pb_glb, Qg, Kg, Vg, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.dO, None, b.A_c, None, b.lse_glb,
                     dQg, dKg, dVg, b.dgate, b.bwd_ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(b.bwd_ws) == 0
    zero = np.zeros_like(d)
    g_loc = oracle.backward_full(c.shape, c.u16("Q"), c.u16("K"), c.u16("V"), zero, c.u16("dO"))
    g_all = oracle.backward_full(c.shape, gu["Q"], gu["K"], gu["V"], d, c.u16("dO"))
    g_loc_g = oracle.backward_full(c.shape, gu["Q"], gu["K"], gu["V"], zero, c.u16("dO"))
    for got, want_, name in zip((dQ, dK, dV), g_loc, ("dQ", "dK", "dV")):
        check_close(to_f64(got), want_, name + " of the local module", outlier_frac=1e-5)
    for got, x, y, name in zip((dQg, dKg, dVg), g_all, g_loc_g, ("dQ", "dK", "dV")):
        check_close(to_f64(got), x - y, name + " of the global module", outlier_frac=1e-5)
    # rows that were not routed get no gradient from the global module: exactly zero
    assert (to_f64(dQg)[d == 0] == 0).all()
    # dgate_t = dO_t . a_t with a_t from the global set (Eq. 7)
    want_gate = (to_f64(b.dO) * ref_glb["a"]).sum(axis=(2, 3)) * d
    check_close(b.dgate.cpu().numpy().astype(np.float64), want_gate, "dgate", 2e-2 * np.sqrt(Hq * D), 2e-3 * np.sqrt(Hq * D))


    # the same layer through the one-call forms: equal to the sequences above (dQ of either set up to the order of its
    # fp32 sums), and with no second set they are l2a_forward / l2a_backward
    two = {k: v.clone() for k, v in dict(O=b.O, S=b.S_save, A=b.A_c, dQ=dQ, dK=dK, dV=dV, dQg=dQg, dKg=dKg, dVg=dVg).items()}
    p = l2a.params(B, L, L, Hq, Hkv, D, W, flags=flags)
    for t in (b.O, dQ, dK, dV, dQg, dKg, dVg):
        t.fill_(float("nan"))
    l2a.l2a_forward_sets(p, b.Q, b.K, b.V, Qg, Kg, Vg, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.O, b.S_save, b.A_c,
                         b.lse_loc, b.lse_glb, b.fwd_ws)
    l2a.l2a_backward_sets(p, b.Q, b.K, b.V, Qg, Kg, Vg, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.dO, b.S_save, b.A_c,
                          b.lse_loc, b.lse_glb, dQ, dK, dV, dQg, dKg, dVg, b.dgate, b.bwd_ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(b.fwd_ws) == 0 and l2a.l2a_workspace_status(b.bwd_ws) == 0
    n = b.n_routed.cpu().numpy()
    for k, got in dict(O=b.O, S=b.S_save, dK=dK, dV=dV, dKg=dKg, dVg=dVg).items():
        assert torch.equal(got.view(torch.int16), two[k].view(torch.int16)), k
    for bi in range(B):
        assert torch.equal(b.A_c[bi, :n[bi]].view(torch.int16), two["A"][bi, :n[bi]].view(torch.int16))
    check_same_or_rounding(dQ, two["dQ"], "dQ (local set)")
    check_same_or_rounding(dQg, two["dQg"], "dQ (global set)")
    c.run_forward()
    want_o = b.O.clone()
    l2a.l2a_forward_sets(c.p, b.Q, b.K, b.V, None, None, None, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.O, b.S_save,
                         b.A_c, b.lse_loc, b.lse_glb, b.fwd_ws)
    torch.cuda.synchronize()
    assert torch.equal(b.O.view(torch.int16), want_o.view(torch.int16))
