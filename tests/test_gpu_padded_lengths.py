"""Sequences of different lengths in one batch, right-padded to a common length.  Causal attention never looks at a
later key, so the rows of a shorter sequence are exactly what a call at its own length gives, and with dO = 0 and
d = 0 on the padding rows (finite padding values) nothing flows back from them into dK, dV."""
import numpy as np
import pytest
import torch

from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import check_same_or_rounding, Case, run_backward

pytestmark = pytest.mark.gpu


def test_right_padded_batch_matches_single_sequences():
    Hq, Hkv, D, W = 4, 2, 128, 200
    lens = (1100, 517)
    L = max(lens)
    singles = []
    for i, n in enumerate(lens):
        d = synth.mask_bernoulli(1, n, 0.3, seed=60 + i)
        c = Case(1, n, Hq, Hkv, D, W, d, seed=70 + i, backward=True)
        c.run_forward()
        run_backward(c)
        singles.append(c)
    d = np.zeros((len(lens), L), np.uint8)
    for i, c in enumerate(singles):
        d[i, :lens[i]] = c.d[0]
    batch = Case(len(lens), L, Hq, Hkv, D, W, d, seed=99, backward=True)
    for name in ("Q", "K", "V", "dO"):
        t = getattr(batch.buf, name)
        t.zero_()                                  # finite padding; dO = 0 there
        for i, c in enumerate(singles):
            t[i, :lens[i]].copy_(getattr(c.buf, name)[0])
    batch.run_forward()
    run_backward(batch)
    for i, c in enumerate(singles):
        n = lens[i]
        for name in ("O", "dQ", "dK", "dV"):
            # bit-identical: same tiles and order of operations per row; a key block may see more query tiles than in
            # the single call, but those are masked or carry dO = 0 and add exact zeros
            got, want = getattr(batch.buf, name)[i, :n], getattr(c.buf, name)[0]
            if name == "dQ":   # summed over the key blocks with fp32 atomics: order not fixed
                check_same_or_rounding(got.contiguous(), want, name)
            else:
                assert torch.equal(got.contiguous().view(torch.int16), want.view(torch.int16)), (name, i)
        assert torch.all(batch.buf.dQ[i, n:] == 0) and torch.all(batch.buf.dK[i, n:] == 0)
        assert torch.all(batch.buf.dV[i, n:] == 0)
