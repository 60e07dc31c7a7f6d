"""Largest case of the suite: one sequence of 2^20 tokens whose Q, O, dO and dQ are 2 GiB each (element offsets
beyond 2^30, byte offsets beyond 2^31), forward + backward, against the oracle on sampled rows and key positions, with
every buffer between pattern-filled guards."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import check_close, to_f64

pytestmark = pytest.mark.gpu


def test_million_token_sequence_forward_and_backward():
    B, L, Hq, Hkv, D, W = 1, 1 << 20, 8, 2, 128, 4096
    seed = 20260317 + 77
    d = synth.mask_clustered(B, L, 0.02, seed)
    assert 0.01 < d.mean() < 0.03
    host = synth.qkv(B, L, Hq, Hkv, D, seed, with_dO=True)
    assert host["Q"].numel() * 2 >= 1 << 31
    p = l2a.params(B, L, L, Hq, Hkv, D, W, flags=l2a.FLAG_SAVE_FOR_BWD)
    buf = l2a.Buffers.allocate(p, backward=True, guard=True)
    for k in ("Q", "K", "V", "dO"):
        getattr(buf, k).copy_(host[k])
    buf.router.copy_(torch.from_numpy(d))
    for t in (buf.O, buf.dQ, buf.dK, buf.dV):
        t.fill_(float("nan"))
    buf.route(l2a.ROUTER_MASK_U8, 0.0)
    buf.forward()
    buf.backward()
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(buf.fwd_ws) == 0 and l2a.l2a_workspace_status(buf.bwd_ws) == 0
    assert buf.check_guards(), "a kernel wrote outside a buffer"
    q_idx, n, prefix = oracle.compact(d)
    assert np.array_equal(buf.q_idx.cpu().numpy(), q_idx) and np.array_equal(buf.n_routed.cpu().numpy(), n)
    assert np.array_equal(buf.prefix.cpu().numpy(), prefix)
    for t in (buf.O, buf.dQ, buf.dK, buf.dV):                      # every element was written
        assert torch.isfinite(t.float()).all()

    sh = oracle.Shape(B, L, L, Hq, Hkv, D, W)
    u16 = {k: synth.as_u16(v) for k, v in host.items()}
    rng = np.random.default_rng(5)
    routed = np.nonzero(d[0])[0]
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 4096, 4097, L // 2, L - 129, L - 128, L - 1],
                                     rng.choice(routed, 20, replace=False), routed[-2:], routed[:2],
                                     rng.choice(L, 16, replace=False)])).astype(np.int32)
    rh = np.repeat(np.arange(Hq, dtype=np.int32), rows.size)
    rt = np.tile(rows, Hq)
    rb = np.zeros_like(rt)
    idx = torch.from_numpy(rows.astype(np.int64)).cuda()

    def by_row(x):
        return x.reshape(Hq, rows.size, D).transpose(1, 0, 2)

    ref = oracle.forward_rows(sh, u16["Q"], u16["K"], u16["V"], d, rb, rh, rt)
    check_close(to_f64(buf.O[0].index_select(0, idx)), by_row(ref["o"]), "O (sampled rows, 1M tokens)")
    check_close(to_f64(buf.S_save[0].index_select(0, idx)), by_row(ref["s"]), "S_save (sampled rows, 1M tokens)")
    want = oracle.dq_rows(sh, u16["Q"], u16["K"], u16["V"], d, u16["dO"], rb, rh, rt)
    check_close(to_f64(buf.dQ[0].index_select(0, idx)), by_row(want), "dQ (sampled rows, 1M tokens)", outlier_frac=1e-5)

    # key positions near the end (the oracle recomputes the soft-max normaliser of every row that sees a key: an early
    # key would cost all 1e10 routed pairs): last block and its edges, window edges, around the last routed burst
    t_r = int(routed[routed < L - 1500][-1])
    js = np.unique(np.concatenate([[L - 4098, L - 4097, L - 1025, L - 1024, L - 129, L - 128, L - 1,
                                    t_r + 1, t_r, t_r - 1, t_r - 127, t_r - 128], rng.choice(np.arange(L - 3000, L), 20, replace=False)])).astype(np.int32)
    jt = torch.from_numpy(js.astype(np.int64)).cuda()
    for g in range(Hkv):
        dk, dv = oracle.dkv_cols(sh, u16["Q"], u16["K"], u16["V"], d, u16["dO"], 0, g, js)
        check_close(to_f64(buf.dK[0].index_select(0, jt)[:, g]), dk, "dK (sampled keys, 1M tokens)", outlier_frac=1e-5)
        check_close(to_f64(buf.dV[0].index_select(0, jt)[:, g]), dv, "dV (sampled keys, 1M tokens)", outlier_frac=1e-5)
