"""The bounded device-side wait: a wait that nothing satisfies runs out after its limit, the CTA records it in the
status word, the host reads L2A_ERR_DEVICE_TIMEOUT, and the context stays usable (no trap, no fault, no endless
loop).  The limit here is a millisecond; the library's kernels use two seconds."""
import time

import pytest
import torch

from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import Case

pytestmark = pytest.mark.gpu


def test_wait_runs_out_and_is_reported_then_work_continues():
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    assert l2a.l2a_workspace_status(ws) == 0
    t0 = time.perf_counter()
    l2a.l2a_selftest_wait_timeout(ws, 1000)
    assert l2a.l2a_workspace_status(ws) == -5          # L2A_ERR_DEVICE_TIMEOUT
    assert time.perf_counter() - t0 < 1.0              # one millisecond of waiting, not a hang
    assert l2a.status_string(-5) not in ("ok", "unknown status")
    # the context is intact: a normal forward runs and its workspace reports no time-out
    d = synth.mask_bernoulli(1, 300, 0.5, seed=1)
    c = Case(1, 300, 2, 1, 128, 64, d, seed=2)
    c.run_forward()
    c.check_forward_full()


def test_selftest_argument_checks():
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    assert l2a.l2a_selftest_wait_timeout(ws, 0, check=False) == -1
    assert l2a.l2a_selftest_wait_timeout(ws, 2_000_000, check=False) == -1
    assert l2a.l2a_selftest_wait_timeout(None, 10, check=False) == -3
