"""Router front and back end around the attention kernels: the one-call layer forward (Eq. 2 -> 3 -> 4 -> 5), the
router's backward under the straight-through estimator (Eq. 7 with the regulariser's gradient), and the attention
backward with a separate gradient for the local output."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import check_same_or_rounding, Case, check_close, run_backward, to_f64

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.cpu().view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("extra", [0, l2a.FLAG_SHARED_WINDOW], ids=["plain", "shared_window"])
def test_forward_routed_equals_the_four_calls(extra):
    B, L, Hq, Hkv, D, W = 2, 1300, 4, 2, 128, 160
    rng = np.random.default_rng(5)
    w = torch.from_numpy((rng.standard_normal(Hq * D) * 0.5).astype(np.float32)).cuda()
    bias = 0.1
    out = {}
    for mode in ("four_calls", "one_call"):
        c = Case(B, L, Hq, Hkv, D, W, np.zeros((B, L), np.uint8), seed=31, backward=True, flags=extra)
        b = c.buf
        logits = torch.empty((B, L), dtype=torch.float32, device="cuda")
        sum_sq = torch.empty((B,), dtype=torch.float32, device="cuda")
        b.O.fill_(float("nan"))
        if mode == "four_calls":
            p1 = l2a.params(B, L, L, Hq, Hkv, D, W, flags=l2a.FLAG_SAVE_FOR_BWD | l2a.FLAG_SKIP_GLOBAL | extra)
            l2a.l2a_forward(p1, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.O, b.S_save, b.A_c,
                            b.lse_loc, b.lse_glb, b.fwd_ws)
            l2a.l2a_router_logits(p1, b.S_save, w, bias, logits, sum_sq)
            l2a.l2a_route_compact(p1, logits, l2a.ROUTER_LOGITS_F32, 0.0, b.d_mask, b.q_idx, b.n_routed, b.prefix,
                                  b.route_ws)
            p2 = l2a.params(B, L, L, Hq, Hkv, D, W, flags=l2a.FLAG_SAVE_FOR_BWD | l2a.FLAG_GLOBAL_PHASE | extra)
            l2a.l2a_forward(p2, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.O, b.S_save, b.A_c,
                            b.lse_loc, b.lse_glb, b.fwd_ws)
        else:
            l2a.l2a_forward_routed(c.p, b.Q, b.K, b.V, w, bias, 0.0, logits, sum_sq, b.d_mask, b.q_idx, b.n_routed,
                                   b.prefix, b.O, b.S_save, b.A_c, b.lse_loc, b.lse_glb, b.route_ws, b.fwd_ws)
        torch.cuda.synchronize()
        assert l2a.l2a_workspace_status(b.fwd_ws) == 0
        out[mode] = dict(O=_bits(b.O), S=_bits(b.S_save), d=b.d_mask.cpu().numpy(), q_idx=b.q_idx.cpu().numpy(),
                         n=b.n_routed.cpu().numpy(), z=logits.cpu().numpy(), case=c)
    a, o = out["four_calls"], out["one_call"]
    for k in ("O", "S", "d", "q_idx", "n", "z"):
        assert np.array_equal(a[k], o[k]), k
    # against the oracle: logits from the oracle's own local output, decisions on the kernel's fp32 logits
    c = o["case"]
    ref0 = oracle.forward_full(c.shape, c.u16("Q"), c.u16("K"), c.u16("V"), np.zeros((B, L), np.uint8))
    z_ref = oracle.router_logits(o["S"], w.cpu().numpy(), bias)
    assert np.abs(o["z"] - z_ref).max() <= 1e-3 * (1 + np.abs(z_ref).max())
    d = oracle.route(o["z"], 0.0)
    assert 0.05 < d.mean() < 0.95
    assert np.array_equal(o["d"], d)
    c.d = d
    ref = c.check_forward_full()
    check_close(to_f64(c.buf.S_save), ref0["s"], "local output")


@pytest.mark.parametrize("B,L,Hq,D,with_dO", [(2, 700, 4, 128, True), (1, 129, 28, 128, True), (3, 64, 2, 64, False)])
def test_router_backward_matches_oracle(B, L, Hq, D, with_dO):
    rng = np.random.default_rng(L)
    t = synth.qkv(B, L, Hq, Hq, D, seed=L, with_dO=True)
    S, dO = t["Q"], t["dO"]                       # any bf16 rows serve as the local output and its gradient
    w = (rng.standard_normal(Hq * D) * 0.3).astype(np.float32)
    z = (rng.standard_normal((B, L)) * 2.0).astype(np.float32)
    dgate = rng.standard_normal((B, L)).astype(np.float32)
    coeff = 0.013
    p = l2a.params(B, L, L, Hq, Hq, D, 16)
    dz = torch.empty((B, L), dtype=torch.float32, device="cuda")
    dw = torch.full((Hq * D,), float("nan"), dtype=torch.float32, device="cuda")
    dbias = torch.full((1,), float("nan"), dtype=torch.float32, device="cuda")
    dS = torch.full((B, L, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda") if with_dO else None
    l2a.l2a_router_backward(p, S.cuda(), torch.from_numpy(w).cuda(), torch.from_numpy(z).cuda(),
                            torch.from_numpy(dgate).cuda(), coeff, dO.cuda() if with_dO else None, dz, dw, dbias, dS)
    torch.cuda.synchronize()
    r_dz, r_dw, r_db, r_dS = oracle.router_backward(synth.as_u16(S), w, z, dgate, coeff,
                                                    synth.as_u16(dO) if with_dO else None)
    # fp32 arithmetic on fp32 inputs: relative 1e-5 on the per-token values, and on the sums relative to the sum of
    # magnitudes of their terms
    assert np.abs(dz.cpu().numpy() - r_dz).max() <= 1e-5 * (1 + np.abs(r_dz).max())
    s64 = to_f64(S).reshape(B, L, -1)
    term_mag = np.einsum("bt,btk->k", np.abs(r_dz), np.abs(s64))
    assert (np.abs(dw.cpu().numpy() - r_dw) <= 1e-5 * (1 + term_mag)).all()
    assert abs(float(dbias.cpu()[0]) - r_db) <= 1e-5 * (1 + np.abs(r_dz).sum())
    if with_dO:
        check_close(to_f64(dS), r_dS, "dS_loc = dO + dz w")


def test_backward_split_is_linear_in_its_two_gradients():
    """dL/ds_t (local branch) and dL/do_t (global branch) enter different parts of the backward; by linearity the
    expected gradients are  bwd(d = 0, dS_loc) + bwd(d, dO) - bwd(d = 0, dO)  from the oracle."""
    B, L, Hq, Hkv, D, W = 2, 900, 4, 2, 128, 128
    d = synth.mask_bernoulli(B, L, 0.3, seed=8)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=44, backward=True)
    c.run_forward()
    b = c.buf
    dS_host = synth.qkv(B, L, Hq, Hkv, D, seed=45, with_dO=True)["dO"]      # an independent bf16 gradient for s_t
    dS_loc = dS_host.cuda()
    for t in (b.dQ, b.dK, b.dV):
        t.fill_(float("nan"))
    l2a.l2a_backward_split(c.p, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.dO, dS_loc, b.S_save, b.A_c,
                           b.lse_loc, b.lse_glb, b.dQ, b.dK, b.dV, b.dgate, b.bwd_ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(b.bwd_ws) == 0
    zero = np.zeros_like(d)
    args = (c.shape, c.u16("Q"), c.u16("K"), c.u16("V"))
    g_loc = oracle.backward_full(*args, zero, synth.as_u16(dS_host))
    g_all = oracle.backward_full(*args, d, c.u16("dO"))
    g_loc_dO = oracle.backward_full(*args, zero, c.u16("dO"))
    for got, name, x, y, z in zip((b.dQ, b.dK, b.dV), ("dQ", "dK", "dV"), g_loc, g_all, g_loc_dO):
        check_close(to_f64(got), x + y - z, name + " (split)", outlier_frac=1e-5)
    # with dS_loc = dO the call is l2a_backward itself (dK, dV bit for bit; dQ up to the order of its fp32 sums)
    first = [_bits(t).copy() for t in (b.dQ, b.dK, b.dV)]
    l2a.l2a_backward_split(c.p, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.dO, b.dO, b.S_save, b.A_c,
                           b.lse_loc, b.lse_glb, b.dQ, b.dK, b.dV, b.dgate, b.bwd_ws)
    torch.cuda.synchronize()
    same = [_bits(t).copy() for t in (b.dQ, b.dK, b.dV)]
    same_dq = b.dQ.clone()
    run_backward(c)
    check_same_or_rounding(same_dq, b.dQ, "dQ")
    for s_, t_ in zip(same[1:], (b.dK, b.dV)):
        assert np.array_equal(s_, _bits(t_))
    assert any(not np.array_equal(f, s_) for f, s_ in zip(first, same))
