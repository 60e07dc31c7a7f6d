import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """How far each GPU-vs-oracle comparison of the session was from the plain 2e-2 bound and from the bound the tests
    apply (tests/gpu_util.py)."""
    try:
        from tests import gpu_util
    except Exception:
        return
    if not gpu_util.STATS:
        return
    agg = {}
    for what, n, n_plain, n_over, ratio in gpu_util.STATS:
        a = agg.setdefault(what, [0, 0, 0, 0, 0.0])
        a[0] += 1; a[1] += n; a[2] += n_plain; a[3] += n_over; a[4] = max(a[4], ratio)
    tr = terminalreporter
    tr.write_sep("-", "parity against the fp64 oracle: elements over the plain bound / over the applied bound")
    for what, (cases, n, n_plain, n_over, ratio) in sorted(agg.items()):
        tr.write_line(f"{what:42s} comparisons {cases:4d}  elements {n:12d}  > 2e-2 (or 1e-3 for lse): {n_plain:6d}  "
                      f"> bound: {n_over:4d}  largest err/bound {ratio:.3f}")
