"""Packed variable-length batches: several sequences back to back on one token axis (l2a_pack_sequences +
l2a_params.seq_bounds).  Expected values: the fp64 oracle run on each sequence by itself."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import Case, EARLY_ROWS, LSE_ABS, check_close, run_backward, to_f64

pytestmark = pytest.mark.gpu


def bounds_of(lengths, total):
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    want = np.empty((total, 2), np.int32)
    for s, e in zip(cu[:-1], cu[1:]):
        want[s:e] = (s, e)
    for t in range(cu[-1], total):          # padding at the end of the axis: sequences of one token
        want[t] = (t, t + 1)
    return cu, want


def packed_case(lengths, Hq, Hkv, D, W, rho, seed, backward=True, flags=0, pad=0):
    total = int(sum(lengths)) + pad
    d = synth.mask_bernoulli(1, total, rho, seed=seed + 1)
    c = Case(1, total, Hq, Hkv, D, W, d, seed=seed, backward=backward, flags=flags)
    cu, want = bounds_of(lengths, total)
    table = l2a.l2a_pack_sequences(torch.from_numpy(cu).cuda(), total)
    torch.cuda.synchronize()
    assert np.array_equal(table.cpu().numpy(), want)
    c.seq_table = table                      # keeps the device table alive
    c.p.seq_bounds = table.data_ptr()
    c.buf.p.seq_bounds = table.data_ptr()
    return c, want


def sequences(want):
    starts = np.unique(want[:, 0])
    return [(int(s), int(want[s, 1])) for s in starts]


def oracle_by_sequence(c, want, backward):
    """Forward (and backward) of every sequence on its own slice; yields (s, e, forward dict, gradients or None)."""
    sh = c.shape
    for s, e in sequences(want):
        n = e - s
        one = oracle.Shape(1, n, n, sh.Hq, sh.Hkv, sh.D, sh.window)
        sl = {k: np.ascontiguousarray(c.u16(k)[:, s:e]) for k in ("Q", "K", "V") + (("dO",) if backward else ())}
        dd = np.ascontiguousarray(c.d[:, s:e])
        fwd = oracle.forward_full(one, sl["Q"], sl["K"], sl["V"], dd)
        grads = oracle.backward_full(one, sl["Q"], sl["K"], sl["V"], dd, sl["dO"]) if backward else None
        yield s, e, fwd, grads


def check_packed(c, want, backward=True):
    b = c.run_forward()
    q_idx, n, prefix = c.check_routing()
    if backward:
        run_backward(c)
    for s, e, fwd, grads in oracle_by_sequence(c, want, backward):
        check_close(to_f64(b.O[:, s:e]), fwd["o"], "O (packed)")
        if backward:
            check_close(to_f64(b.S_save[:, s:e]), fwd["s"], "S_save (packed)")
            check_close(to_f64(b.lse_loc[:, :, s:e]), fwd["lse_loc"], "lse_loc", LSE_ABS, LSE_ABS)
            c0, c1 = int(prefix[0, s]), int(prefix[0, e])            # the sequence's compact rows
            rows = q_idx[0, c0:c1] - s
            if c1 > c0:
                check_close(to_f64(b.A_c[:, c0:c1]), fwd["a"][:, rows], "A_c (packed)")
                check_close(to_f64(b.lse_glb[:, :, c0:c1]), fwd["lse_glb"][:, :, rows], "lse_glb", LSE_ABS, LSE_ABS)
            for got, ref, name in zip((b.dQ, b.dK, b.dV), grads, ("dQ", "dK", "dV")):
                check_close(to_f64(got[:, s:e]), ref, name + " (packed)", outlier_frac=1e-5, early_rows=EARLY_ROWS)


@pytest.mark.parametrize("lengths,Hq,Hkv,D,W,rho,pad", [
    ([300, 1, 129, 700, 128, 513, 5], 4, 2, 128, 150, 0.3, 0),     # boundaries inside tiles, on tile edges, a single token
    ([256, 256, 384], 2, 1, 128, 64, 0.5, 0),                      # every boundary on a tile edge
    ([77, 1000, 3], 2, 2, 64, 2000, 0.25, 0),                      # window longer than any sequence: local = causal
    ([500, 260], 2, 1, 128, 0, 1.0, 0),                            # W = 0, every token routed
    ([130, 400], 4, 1, 64, 100, 0.0, 0),                           # nothing routed
    ([600, 200], 2, 1, 128, 90, 0.4, 100),                         # padding after the last sequence
])
def test_packed_batch_equals_one_call_per_sequence(lengths, Hq, Hkv, D, W, rho, pad):
    c, want = packed_case(lengths, Hq, Hkv, D, W, rho, seed=700 + len(lengths) + W, pad=pad)
    assert len(sequences(want)) == len(lengths) + pad
    check_packed(c, want)


def test_packed_batch_with_shared_window_and_forward_only():
    lengths = [333, 900, 128, 250]
    c, want = packed_case(lengths, 4, 2, 128, 100, 0.35, seed=733, flags=l2a.FLAG_SHARED_WINDOW)
    check_packed(c, want)
    c, want = packed_case(lengths, 4, 2, 128, 100, 0.35, seed=734, backward=False)
    check_packed(c, want, backward=False)


def test_packed_batch_many_sequences_long_axis():
    # 16K tokens: sequences from 100 to 6144 tokens, window shorter and longer than them
    lengths = [4096, 2048, 6144, 100, 3996]
    c, want = packed_case(lengths, 4, 2, 128, 2048, 0.2, seed=741)
    check_packed(c, want)


def test_packed_rejects_what_it_does_not_cover():
    table = l2a.l2a_pack_sequences(torch.tensor([0, 100, 256], dtype=torch.int32, device="cuda"), 256)
    for kw in (dict(B=2, Lq=256, Lk=256), dict(B=1, Lq=256, Lk=512)):
        p = l2a.params(kw["B"], kw["Lq"], kw["Lk"], 2, 1, 128, 16, seq_bounds=table)
        with pytest.raises(l2a.L2AError) as e:
            l2a.l2a_workspace_bytes(p)
        assert e.value.code == -1


def test_packed_batch_with_global_attention_for_every_token():
    """Forced-global iterations (Section 3.3) on a packed batch: a_t of every token comes from its own sequence."""
    lengths = [200, 515, 129, 300]
    c, want = packed_case(lengths, 4, 2, 128, 80, 0.3, seed=751, flags=l2a.FLAG_FORCE_ALL_GLOBAL)
    b = c.run_forward()
    run_backward(c)
    sh = c.shape
    for s, e, fwd, grads in oracle_by_sequence(c, want, True):
        n = e - s
        one = oracle.Shape(1, n, n, sh.Hq, sh.Hkv, sh.D, sh.window)
        sl = {k: np.ascontiguousarray(c.u16(k)[:, s:e]) for k in ("Q", "K", "V", "dO")}
        every = oracle.forward_full(one, sl["Q"], sl["K"], sl["V"], np.ones((1, n), np.uint8))
        check_close(to_f64(b.O[:, s:e]), fwd["o"], "O (packed, forced global)")
        check_close(to_f64(b.A_c[:, s:e]), every["a"], "A by row (packed)")
        check_close(to_f64(b.lse_glb[:, :, s:e]), every["lse_glb"], "lse_glb by row", LSE_ABS, LSE_ABS)
        for got, ref, name in zip((b.dQ, b.dK, b.dV), grads, ("dQ", "dK", "dV")):
            check_close(to_f64(got[:, s:e]), ref, name + " (packed, forced global)", outlier_frac=1e-5, early_rows=EARLY_ROWS)
        rt = np.arange(n)
        gate = oracle.dgate_rows(one, sl["Q"], sl["K"], sl["V"], sl["dO"], np.zeros_like(rt), rt)
        check_close(to_f64(b.dgate[:, s:e]), gate.reshape(1, n), "dgate (packed, every token)", 5e-2, 5e-3)
