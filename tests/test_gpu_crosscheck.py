"""Cross-check against an unrelated implementation: with every token routed and a window that covers the whole
prefix, both modules are plain causal attention, so o = 2 * causal_attention(Q, K, V).  PyTorch's own fp32 attention
(explicit soft-max on the GPU, autograd for the gradients) stands in for it on every element of a 4096-token layer
with grouped heads.  The oracle remains the reference of record; this guards against an error shared by the oracle's
pins and the kernels' author."""
import numpy as np
import pytest
import torch

from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import Case, check_close, run_backward, to_f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("extra", [0, l2a.FLAG_SHARED_WINDOW], ids=["plain", "shared_window"])
def test_all_routed_full_window_is_twice_causal_attention(extra):
    B, L, Hq, Hkv, D = 1, 4096, 8, 2, 128
    d = np.ones((B, L), np.uint8)
    c = Case(B, L, Hq, Hkv, D, L, d, seed=21, backward=True, flags=extra)
    c.run_forward()
    run_backward(c)
    b = c.buf
    G = Hq // Hkv
    q = b.Q.float().permute(0, 2, 1, 3).detach().requires_grad_(True)                       # [B, Hq, L, D]
    k = b.K.float().permute(0, 2, 1, 3).detach().requires_grad_(True)                       # [B, Hkv, L, D]
    v = b.V.float().permute(0, 2, 1, 3).detach().requires_grad_(True)
    scores = torch.einsum("bhld,bhmd->bhlm", q, k.repeat_interleave(G, dim=1)) / D ** 0.5
    mask = torch.ones(L, L, dtype=torch.bool, device="cuda").tril()
    p = torch.softmax(scores.masked_fill(~mask, float("-inf")), dim=-1)
    o = 2.0 * torch.einsum("bhlm,bhmd->bhld", p, v.repeat_interleave(G, dim=1))
    o.backward(b.dO.float().permute(0, 2, 1, 3))
    back = lambda t: to_f64(t.permute(0, 2, 1, 3))
    check_close(to_f64(b.O), back(o.detach()), "O vs PyTorch")
    check_close(to_f64(b.dQ), back(q.grad), "dQ vs PyTorch", outlier_frac=1e-5)
    check_close(to_f64(b.dK), back(k.grad), "dK vs PyTorch", outlier_frac=1e-5)
    check_close(to_f64(b.dV), back(v.grad), "dV vs PyTorch", outlier_frac=1e-5)
