"""Strided inputs and outputs (slices of a fused QKV projection buffer; O, dO and the gradients inside wider
buffers): the same kernels on the same values, so the results must equal the dense run bit for bit, and the bytes
between the rows must stay untouched."""
import numpy as np
import pytest
import torch

from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import check_same_or_rounding, Case, run_backward

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.contiguous().view(torch.int16)


@pytest.mark.parametrize("extra", [0, l2a.FLAG_SHARED_WINDOW], ids=["plain", "shared_window"])
@pytest.mark.parametrize("B,L,Hq,Hkv,D,W", [(2, 700, 4, 2, 128, 100), (1, 1300, 6, 2, 64, 300)])
def test_strided_tensors_match_dense(B, L, Hq, Hkv, D, W, extra):
    d = synth.mask_bernoulli(B, L, 0.3, seed=5)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=77, backward=True, flags=extra)
    c.run_forward()
    run_backward(c)
    b = c.buf
    dense = {k: getattr(b, k).clone() for k in ("O", "S_save", "dQ", "dK", "dV", "dgate", "lse_loc")}

    # fused [B, L + 3, (Hq + 2 Hkv) D + 16] buffers: Q | K | V slices of one, dQ | dK | dV slices of another
    wq, wk = Hq * D, Hkv * D
    tok = wq + 2 * wk + 16
    Lpad = L + 3
    fused = torch.full((B, Lpad, tok), float("nan"), dtype=torch.bfloat16, device="cuda")
    grads = torch.full((B, Lpad, tok), 7.0, dtype=torch.bfloat16, device="cuda")
    fused[:, :L, :wq] = b.Q.view(B, L, wq)
    fused[:, :L, wq:wq + wk] = b.K.view(B, L, wk)
    fused[:, :L, wq + wk:wq + 2 * wk] = b.V.view(B, L, wk)
    Q, K, V = fused[:, :, :wq], fused[:, :, wq:wq + wk], fused[:, :, wq + wk:]
    dQ, dK, dV = grads[:, :, :wq], grads[:, :, wq:wq + wk], grads[:, :, wq + wk:]
    # O and dO live in buffers with a wider token pitch
    opitch = wq + 24
    Obuf = torch.full((B, L, opitch), 5.0, dtype=torch.bfloat16, device="cuda")
    dObuf = torch.zeros((B, L, opitch), dtype=torch.bfloat16, device="cuda")
    dObuf[:, :, :wq] = b.dO.view(B, L, wq)
    st = (Lpad * tok, tok)
    p = l2a.params(B, L, L, Hq, Hkv, D, W, flags=l2a.FLAG_SAVE_FOR_BWD | extra, q_stride=st, k_stride=st, v_stride=st,
                   o_stride=(L * opitch, opitch))
    b.S_save.fill_(float("nan"))
    l2a.l2a_forward(p, Q, K, V, b.d_mask, b.q_idx, b.n_routed, b.prefix, Obuf, b.S_save, b.A_c, b.lse_loc, b.lse_glb,
                    b.fwd_ws)
    l2a.l2a_backward(p, Q, K, V, b.d_mask, b.q_idx, b.n_routed, b.prefix, dObuf, b.S_save, b.A_c, b.lse_loc,
                     b.lse_glb, dQ, dK, dV, b.dgate, b.bwd_ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(b.fwd_ws) == 0 and l2a.l2a_workspace_status(b.bwd_ws) == 0
    assert torch.equal(_bits(Obuf[:, :, :wq]), _bits(dense["O"].view(B, L, wq)))
    assert torch.equal(_bits(b.S_save), _bits(dense["S_save"]))
    assert torch.equal(b.lse_loc, dense["lse_loc"])
    check_same_or_rounding(dQ[:, :L], dense["dQ"].view(B, L, wq), "dQ")   # fp32 atomic sums: order not fixed
    assert torch.equal(_bits(dK[:, :L]), _bits(dense["dK"].view(B, L, wk)))
    assert torch.equal(_bits(dV[:, :L, :wk]), _bits(dense["dV"].view(B, L, wk)))
    assert torch.equal(b.dgate, dense["dgate"])
    # nothing outside the addressed rows and columns was written
    assert (Obuf[:, :, wq:] == 5.0).all()
    assert (grads[:, L:] == 7.0).all() and (grads[:, :, wq + 2 * wk:] == 7.0).all()


def test_strided_cache_in_decode():
    B, Lk, Hq, Hkv, D, W = 3, 3000, 8, 2, 128, 256
    t = synth.qkv(B, 1, Hq, Hkv, D, seed=4, Lk=Lk)
    d = torch.tensor([1, 0, 1], dtype=torch.uint8, device="cuda")
    p = l2a.params(B, 1, Lk, Hq, Hkv, D, W)
    ws = torch.empty(l2a.l2a_decode_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    O = torch.empty((B, 1, Hq, D), dtype=torch.bfloat16, device="cuda")
    q, K, V = (t[k].cuda() for k in ("Q", "K", "V"))
    l2a.l2a_decode(p, q, K, V, d, O, ws)
    # the same cache as K | V slices of one buffer allocated for 4096 positions
    wk = Hkv * D
    cache = torch.full((B, 4096, 2 * wk), float("nan"), dtype=torch.bfloat16, device="cuda")
    cache[:, :Lk, :wk] = K.view(B, Lk, wk)
    cache[:, :Lk, wk:] = V.view(B, Lk, wk)
    st = (4096 * 2 * wk, 2 * wk)
    ps = l2a.params(B, 1, Lk, Hq, Hkv, D, W, k_stride=st, v_stride=st)
    O2 = torch.empty_like(O)
    l2a.l2a_decode(ps, q, cache[:, :, :wk], cache[:, :, wk:], d, O2, ws)
    torch.cuda.synchronize()
    assert torch.equal(O.view(torch.int16), O2.view(torch.int16))
