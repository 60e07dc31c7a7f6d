"""The allocation-free routing entry point against the regular one.

``l2a_route_compact_static`` serves callers that have no way to get device scratch memory at call time
(an engine whose pools already own the whole GPU, a plug-in that receives tensors but no allocator, a
loop that must stay clear of cudaMalloc).  Its scratch is a fixed array inside the library, shared by all
calls, so the test makes two calls in a row with different inputs and requires each to match what
``l2a_route_compact`` (caller-provided workspace) produces for the same input: integer results, bit exact.
This file sorts last on purpose so that a run stopping at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2603_17484_b200 import l2a, synth

pytestmark = pytest.mark.gpu


def _outputs(B, L):
    dev = "cuda"
    return (torch.full((B, L), 77, dtype=torch.uint8, device=dev), torch.full((B, L), -5, dtype=torch.int32, device=dev),
            torch.full((B,), -5, dtype=torch.int32, device=dev), torch.full((B, L + 1), -5, dtype=torch.int32, device=dev))


def _same(a, b):
    return all(torch.equal(x, y) for x, y in zip(a, b))


def test_static_scratch_route_matches_workspace_route_twice():
    B, L = 3, 50001
    p = l2a.params(B, L, L, 4, 2, 128, 64)
    r_bytes, _, _ = l2a.l2a_workspace_bytes(p)
    ws = torch.empty(r_bytes, dtype=torch.uint8, device="cuda")
    # call 1: uint8 mask, dense routing; call 2: fp32 logits, sparse routing -> the shared scratch holds
    # larger stale counts from call 1 when call 2 runs
    mask = torch.from_numpy(synth.mask_bernoulli(B, L, 0.7, seed=11)).cuda()
    logits = torch.from_numpy(synth.router_logits(B, L, -2.0, seed=12)).cuda()
    for router, kind, thr in ((mask, l2a.ROUTER_MASK_U8, 0.0), (logits, l2a.ROUTER_LOGITS_F32, 0.0)):
        want, got = _outputs(B, L), _outputs(B, L)
        l2a.l2a_route_compact(p, router, kind, thr, *want, ws)
        l2a.l2a_route_compact_static(p, router, kind, thr, *got)
        torch.cuda.synchronize()
        assert _same(got, want)
        assert int(got[2].sum()) > 0


def test_static_scratch_route_rejects_oversized_shapes_on_the_host():
    # 4097 batch rows x 1 block each exceed the 4096 fixed slots: refused before any launch
    B, L = 4097, 8
    p = l2a.params(B, L, L, 1, 1, 64, 1)
    outs = _outputs(B, L)
    router = torch.zeros((B, L), dtype=torch.uint8, device="cuda")
    assert l2a.l2a_route_compact_static(p, router, l2a.ROUTER_MASK_U8, 0.0, *outs, check=False) == -2
    torch.cuda.synchronize()
    assert int(outs[2][0]) == -5   # untouched
