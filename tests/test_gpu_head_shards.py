"""Head-parallel sharding needs no exchange on the attention path: a rank that owns the KV heads [g0, g1) and their
query heads calls the same entry points on slices of the tensors (the head stride stays D, the token stride is the
full row), and gets exactly the columns the whole call writes.  Run here as two shards on one GPU."""
import numpy as np
import pytest
import torch

from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import check_same_or_rounding, Case, run_backward

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("extra", [0, l2a.FLAG_SHARED_WINDOW], ids=["plain", "shared_window"])
def test_two_head_shards_equal_the_whole_layer(extra):
    B, L, Hq, Hkv, D, W = 2, 900, 8, 4, 128, 160
    d = synth.mask_bernoulli(B, L, 0.3, seed=11)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=13, backward=True, flags=extra)
    c.run_forward()
    run_backward(c, with_dgate=True)
    b = c.buf
    whole = {k: getattr(b, k).clone() for k in ("O", "dQ", "dK", "dV", "dgate")}
    n_shards = 2
    hq, hkv = Hq // n_shards, Hkv // n_shards
    out = {k: torch.full_like(whole[k], float("nan")) for k in ("O", "dQ", "dK", "dV")}
    dgate = torch.zeros_like(whole["dgate"])
    qs, ks = (L * Hq * D, Hq * D), (L * Hkv * D, Hkv * D)
    p = l2a.params(B, L, L, hq, hkv, D, W, flags=l2a.FLAG_SAVE_FOR_BWD | extra, q_stride=qs, k_stride=ks, v_stride=ks,
                   o_stride=qs)
    sizes = l2a.l2a_workspace_bytes(p)
    fwd_ws = torch.empty(sizes[1], dtype=torch.uint8, device="cuda")
    bwd_ws = torch.empty(sizes[2], dtype=torch.uint8, device="cuda")
    S = torch.empty((B, L, hq, D), dtype=torch.bfloat16, device="cuda")
    A = torch.empty_like(S)
    lse_loc = torch.empty((B, hq, L), dtype=torch.float32, device="cuda")
    lse_glb = torch.empty_like(lse_loc)
    part = torch.empty((B, L), dtype=torch.float32, device="cuda")
    for r in range(n_shards):
        q0, k0 = r * hq, r * hkv
        Q, K, V, dO = b.Q[:, :, q0:], b.K[:, :, k0:], b.V[:, :, k0:], b.dO[:, :, q0:]
        O, dQ, dK, dV = out["O"][:, :, q0:], out["dQ"][:, :, q0:], out["dK"][:, :, k0:], out["dV"][:, :, k0:]
        l2a.l2a_forward(p, Q, K, V, b.d_mask, b.q_idx, b.n_routed, b.prefix, O, S, A, lse_loc, lse_glb, fwd_ws)
        l2a.l2a_backward(p, Q, K, V, b.d_mask, b.q_idx, b.n_routed, b.prefix, dO, S, A, lse_loc, lse_glb, dQ, dK, dV,
                         part, bwd_ws)
        torch.cuda.synchronize()
        assert l2a.l2a_workspace_status(fwd_ws) == 0 and l2a.l2a_workspace_status(bwd_ws) == 0
        dgate += part      # the gate gradient sums over heads: the one value ranks would have to add up
    for k in out:
        if k == "dQ":      # summed over the key blocks with fp32 atomics: order not fixed
            check_same_or_rounding(out[k], whole[k], k)
        else:
            assert torch.equal(out[k].view(torch.int16), whole[k].view(torch.int16)), k
    assert torch.allclose(dgate, whole["dgate"], rtol=1e-5, atol=1e-4)
