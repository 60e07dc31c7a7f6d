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


@pytest.mark.parametrize("B,L,backward", [(1, 4389, True), (2, 1300, True), (1, 4389, False)])
def test_pipelined_steps_on_alternating_buffers_match_blocking_steps(B, L, backward):
    """Five steps enqueued with l2a_step_host_async on two alternating sets of device tensors, with two different input
    sets taking turns, each step's results in host buffers of its own: every step equals the blocking call on the same
    inputs (a step that read or overwrote the other step's tensors too early would not)."""
    Hq, Hkv, D, W = 4, 2, 128, 256
    cases, hosts, want = [], [], []
    for k, seed in enumerate((31, 47)):
        d = synth.mask_bernoulli(B, L, 0.25 + 0.1 * k, seed=seed)
        c = Case(B, L, Hq, Hkv, D, W, d, seed=seed + 5, backward=backward)
        h = {n: v.pin_memory() for n, v in c.host.items()}
        h["router"] = torch.from_numpy(d).pin_memory()
        names = ("O", "dQ", "dK", "dV") if backward else ("O",)
        for n in names:
            h[n] = torch.empty_like(getattr(c.buf, n), device="cpu").pin_memory()
        l2a.l2a_step_host(c.p, h, c.buf, l2a.ROUTER_MASK_U8, 0.0)                 # blocking reference
        want.append({n: h[n].clone() for n in names})
        cases.append(c); hosts.append(h)
    outs = []
    for step in range(5):
        k = step & 1                       # inputs k on device set k
        h = dict(hosts[k])
        for n in names:
            h[n] = torch.full_like(hosts[k][n], float("nan")).pin_memory()
        # poison the device inputs of this set from the host side of the stream order: the step must upload them itself
        l2a.l2a_step_host_async(cases[k].p, h, cases[k].buf, l2a.ROUTER_MASK_U8, 0.0)
        outs.append((k, h))
    l2a.l2a_step_host_wait()
    for c in cases:
        assert l2a.l2a_workspace_status(c.buf.fwd_ws) == 0
        assert not backward or l2a.l2a_workspace_status(c.buf.bwd_ws) == 0
        assert c.buf.check_guards()
    for step, (k, h) in enumerate(outs):
        for n in names:
            if n == "dQ":
                check_same_or_rounding(h["dQ"], want[k]["dQ"], f"dQ of pipelined step {step}")
            else:
                assert torch.equal(h[n].view(torch.int16), want[k][n].view(torch.int16)), (step, n)
    # a blocking step while pipelined steps are pending is refused; after the wait it works again
    l2a.l2a_step_host_async(cases[0].p, hosts[0], cases[0].buf, l2a.ROUTER_MASK_U8, 0.0)
    assert l2a.l2a_step_host(cases[1].p, hosts[1], cases[1].buf, l2a.ROUTER_MASK_U8, 0.0, check=False) == -1
    l2a.l2a_step_host_wait()
    l2a.l2a_step_host(cases[1].p, hosts[1], cases[1].buf, l2a.ROUTER_MASK_U8, 0.0)
