"""L2A_FLAG_SHARED_WINDOW: Global Attention of a routed row covers only the keys before its window and is merged
with the local result (the shared-projection variant of the paper's ablations).  The layer's outputs mean the same,
so the bar is the same parity against the fp64 oracle, forward and backward."""
import numpy as np
import pytest
import torch

from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import check_same_or_rounding, Case, check_backward_full, check_close, run_backward, to_f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,Lq,Lk,Hq,Hkv,D,W,rho", [
    (1, 700, 700, 2, 1, 128, 200, 0.3),      # tiles with and without keys before the window
    (2, 513, 513, 4, 2, 128, 128, 0.5),
    (1, 300, 1000, 2, 2, 64, 96, 0.4),       # queries are the last rows of a longer key sequence
    (1, 1500, 1500, 8, 2, 128, 256, 0.1),
    (1, 400, 400, 2, 1, 128, 4096, 1.0),     # window longer than the sequence: the global pass has no key at all
    (1, 900, 900, 2, 1, 64, 300, 0.0),       # nothing routed
    (1, 1000, 1000, 1, 1, 128, 0, 0.5),      # W = 0: the window is the token itself
    (1, 1300, 1300, 2, 2, 128, 127, 1.0),    # all routed, window edge one short of a key block
    (1, 1, 1, 1, 1, 128, 4, 1.0),
    (1, 300, 300, 2, 1, 128, 2 ** 31 - 1, 0.5),   # the largest window the ABI accepts
])
def test_shared_window_forward_backward(B, Lq, Lk, Hq, Hkv, D, W, rho):
    d = synth.mask_bernoulli(B, Lq, rho, seed=Lq + W)
    c = Case(B, Lq, Hq, Hkv, D, W, d, seed=Lq + 5 * D, Lk=Lk, backward=True, flags=l2a.FLAG_SHARED_WINDOW)
    c.buf.A_c.fill_(float("nan"))
    c.buf.lse_glb.fill_(float("nan"))
    c.run_forward()
    c.check_forward_full()
    run_backward(c)
    check_backward_full(c)


def test_shared_window_matches_plain_forward():
    """Same inputs with and without the flag: the two O differ by rounding only."""
    B, L, Hq, Hkv, D, W = 1, 2100, 4, 2, 128, 512
    d = synth.mask_bernoulli(B, L, 0.3, seed=77)
    plain = Case(B, L, Hq, Hkv, D, W, d, seed=12, backward=True)
    plain.run_forward()
    fused = Case(B, L, Hq, Hkv, D, W, d, seed=12, backward=True, flags=l2a.FLAG_SHARED_WINDOW)
    fused.run_forward()
    assert torch.equal(plain.buf.S_save.view(torch.int16), fused.buf.S_save.view(torch.int16))
    assert torch.equal(plain.buf.lse_loc, fused.buf.lse_loc)
    check_close(to_f64(fused.buf.O), to_f64(plain.buf.O), "O shared-window vs plain")
    n = int(plain.buf.n_routed[0])
    check_close(to_f64(fused.buf.lse_glb[:, :, :n]), to_f64(plain.buf.lse_glb[:, :, :n]), "lse_glb", 2e-3, 2e-4)


def test_shared_window_without_saving():
    """Inference call (no L2A_FLAG_SAVE_FOR_BWD): lse_loc is still needed and is the only extra buffer."""
    B, L, Hq, Hkv, D, W = 1, 1100, 2, 1, 128, 256
    d = synth.mask_bernoulli(B, L, 0.4, seed=3)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=31, backward=False, flags=l2a.FLAG_SHARED_WINDOW)
    b = c.buf
    b.route(c.kind, c.threshold)
    assert l2a.l2a_forward(c.p, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.O, None, None, None, None,
                           b.fwd_ws, check=False) == -1  # L2A_ERR_INVALID_ARG
    lse_loc = torch.empty(B, Hq, L, dtype=torch.float32, device="cuda")
    b.O.fill_(float("nan"))
    l2a.l2a_forward(c.p, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.O, None, None, lse_loc, None,
                    b.fwd_ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(b.fwd_ws) == 0
    ref = c.oracle_forward()
    check_close(to_f64(b.O), ref["o"], "O")


def test_shared_window_rejects_other_modes():
    d = synth.mask_bernoulli(1, 300, 0.5, seed=4)
    for extra in (l2a.FLAG_SKIP_LOCAL, l2a.FLAG_FORCE_ALL_GLOBAL):
        c = Case(1, 300, 2, 1, 128, 64, d, seed=8, backward=(extra == l2a.FLAG_FORCE_ALL_GLOBAL),
                 flags=l2a.FLAG_SHARED_WINDOW | extra)
        b = c.buf
        b.route(c.kind, c.threshold)
        code = l2a.l2a_forward(c.p, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.O, b.S_save, b.A_c,
                               b.lse_loc, b.lse_glb, b.fwd_ws, check=False)
        assert code == -1  # L2A_ERR_INVALID_ARG


@pytest.mark.parametrize("backward", [False, True])
def test_shared_window_step_host_and_routed_forward(backward):
    """The host-buffer step (row-range path) and l2a_forward_routed pass the flag on: bit-identical to l2a_forward."""
    B, L, Hq, Hkv, D, W = 1, 4389, 4, 2, 128, 256
    d = synth.mask_bernoulli(B, L, 0.3, seed=17)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=23, backward=backward, flags=l2a.FLAG_SHARED_WINDOW)
    if not backward:
        c.buf.lse_loc = torch.empty(B, Hq, L, dtype=torch.float32, device="cuda")
    c.run_forward()
    want = {"O": c.buf.O.clone()}
    if backward:
        run_backward(c)
        want.update(dQ=c.buf.dQ.clone(), dK=c.buf.dK.clone(), dV=c.buf.dV.clone())
    host = {k: v.pin_memory() for k, v in c.host.items()}
    host["router"] = torch.from_numpy(d).pin_memory()
    for k, w in want.items():
        host[k] = torch.empty_like(w, device="cpu").pin_memory()
        getattr(c.buf, k).zero_()
    l2a.l2a_step_host(c.p, host, c.buf, l2a.ROUTER_MASK_U8, 0.0)
    for k, w in want.items():
        if k == "dQ":      # summed over the key blocks with fp32 atomics: order not fixed
            check_same_or_rounding(host[k], w.cpu(), k)
        else:
            assert torch.equal(host[k].view(torch.int16), w.cpu().view(torch.int16)), k


def test_shared_window_split_backward_falls_back():
    """With a separate gradient for the local output the two modules no longer share dP: the backward ignores the
    flag there, bit-identical to the call without it."""
    B, L, Hq, Hkv, D, W = 1, 900, 2, 1, 128, 200
    d = synth.mask_bernoulli(B, L, 0.4, seed=6)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=41, backward=True)
    c.run_forward()
    run_backward(c)
    want = {k: getattr(c.buf, k).clone() for k in ("dQ", "dK", "dV")}
    b = c.buf
    p = l2a.params(B, L, L, Hq, Hkv, D, W, flags=l2a.FLAG_SAVE_FOR_BWD | l2a.FLAG_SHARED_WINDOW)
    dS_loc = b.dO.clone()
    for t in (b.dQ, b.dK, b.dV):
        t.fill_(float("nan"))
    l2a.l2a_backward_split(p, b.Q, b.K, b.V, b.d_mask, b.q_idx, b.n_routed, b.prefix, b.dO, dS_loc, b.S_save, b.A_c,
                           b.lse_loc, b.lse_glb, b.dQ, b.dK, b.dV, None, b.bwd_ws)
    torch.cuda.synchronize()
    for k, w in want.items():
        if k == "dQ":
            check_same_or_rounding(getattr(b, k), w, k)
        else:
            assert torch.equal(getattr(b, k).view(torch.int16), w.view(torch.int16)), k
