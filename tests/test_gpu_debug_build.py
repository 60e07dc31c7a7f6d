"""The index-checking build of the library (-DL2A_DEBUG, libl2a_debug.so): every index derived from q_idx / prefix /
tile metadata is checked against its tensor before a store; a violation is reported through the workspace status word
(L2A_ERR_DEVICE_BOUNDS) and the store is skipped.  With the pattern-filled guards around every buffer this stands in
for a memory checker.  The checks run in a child process so that this session keeps the normal library loaded."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import numpy as np, torch
from paper_2603_17484_b200 import build, l2a, synth
l2a.LIB_PATH = build.build_lib(debug=True)
assert "debug" in l2a.version()
from tests.gpu_util import Case, check_backward_full, run_backward

# 1. correct inputs: no check fires, results match the oracle, nothing is written outside a buffer
for (B, Lq, Lk, Hq, Hkv, D, W, rho, flags) in [(1, 700, 700, 2, 1, 128, 200, 0.3, 0), (2, 513, 513, 4, 2, 128, 128, 0.5, 0),
                                                 (1, 300, 1000, 2, 2, 64, 96, 0.4, 0), (1, 1500, 1500, 4, 2, 128, 256, 0.1, 64),
                                                 (1, 129, 129, 1, 1, 128, 16, 1.0, 0), (1, 900, 900, 2, 1, 64, 300, 0.0, 0)]:
    d = synth.mask_bernoulli(B, Lq, rho, seed=Lq + W)
    c = Case(B, Lq, Hq, Hkv, D, W, d, seed=Lq + 3 * D, Lk=Lk, backward=True, flags=flags)
    c.run_forward()
    c.check_forward_full()
    run_backward(c)
    check_backward_full(c)

# 1b. a packed variable-length batch: the same checks with per-sequence masks, tile ranges and item lists
from tests.test_gpu_packed import packed_case, check_packed
c, want = packed_case([300, 1, 129, 450], 4, 2, 128, 100, 0.4, seed=77)
check_packed(c, want)

# 2. a compact index one past the end: reported, the row is not stored, the guards stay intact
B, L, Hq, Hkv, D, W = 1, 600, 2, 1, 128, 64
d = synth.mask_bernoulli(B, L, 0.3, seed=4)
c = Case(B, L, Hq, Hkv, D, W, d, seed=8, backward=True)
b = c.buf
b.route(c.kind, 0.0)
n = int(b.n_routed[0])
b.q_idx[0, n - 1] = L
b.forward()
torch.cuda.synchronize()
assert l2a.l2a_workspace_status(b.fwd_ws) == -6, l2a.l2a_workspace_status(b.fwd_ws)
assert b.check_guards()
print("DEBUG_BUILD_OK")
"""


def test_debug_build_checks_indices():
    r = subprocess.run([sys.executable, "-c", CHILD, ROOT], cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "DEBUG_BUILD_OK" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
