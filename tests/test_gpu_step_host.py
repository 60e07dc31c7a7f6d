"""The host-buffer entry point (copies overlapped with the kernels) gives the same results as the device-buffer calls."""
import numpy as np
import pytest
import torch

from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import check_same_or_rounding, Case, run_backward

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("backward", [False, True])
# one long sequence takes the path that uploads K, V and Q in row ranges and starts the attention of each range as
# it lands; the last case has more keys than queries (q_pos_offset = 300)
@pytest.mark.parametrize("B,L,Lk", [(2, 1300, None), (1, 4389, None), (1, 4200, 4500)])
def test_step_host_matches_device_calls(backward, B, L, Lk):
    Hq, Hkv, D, W = 4, 2, 128, 256
    d = synth.mask_bernoulli(B, L, 0.3, seed=17)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=23, backward=backward, Lk=Lk)
    c.run_forward()
    want = {"O": c.buf.O.clone()}
    if backward:
        run_backward(c)
        want.update(dQ=c.buf.dQ.clone(), dK=c.buf.dK.clone(), dV=c.buf.dV.clone())
    host = {k: v.pin_memory() for k, v in c.host.items()}
    host["router"] = torch.from_numpy(d).pin_memory()
    for k in want:
        host[k] = torch.empty_like(want[k], device="cpu").pin_memory()
    for t in (c.buf.Q, c.buf.K, c.buf.V, c.buf.O):
        t.zero_()
    for rep in range(2):            # twice: the helper streams and events are reused
        for k in want:
            host[k].fill_(float("nan"))
        l2a.l2a_step_host(c.p, host, c.buf, l2a.ROUTER_MASK_U8, 0.0)
        for k, w in want.items():
            if k == "dQ":      # summed over the key blocks with fp32 atomics: order not fixed
                check_same_or_rounding(host[k], w.cpu(), k)
            else:
                assert torch.equal(host[k].view(torch.int16), w.cpu().view(torch.int16)), (k, rep)
