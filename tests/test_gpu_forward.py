"""GPU parity: routing/compaction bit-exact, forward outputs against the fp64 oracle (all through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import Case, check_close, to_f64, LSE_ABS

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------------------- routing / compaction

@pytest.mark.parametrize("B,L,rho", [(1, 1, 1.0), (1, 1, 0.0), (2, 37, 0.3), (3, 4096, 0.5), (2, 4097, 0.9),
                                      (1, 10000, 0.01), (1, 131072, 0.2), (4, 8191, 1.0), (2, 5000, 0.0)])
def test_route_compact_mask_bit_exact(B, L, rho):
    d = synth.mask_bernoulli(B, L, rho, seed=L + B)
    p = l2a.params(B, L, L, 4, 2, 128, 16)
    buf = l2a.Buffers.allocate(p)
    buf.q_idx.fill_(12345); buf.prefix.fill_(-7)
    buf.router.copy_(torch.from_numpy(d))
    buf.route()
    torch.cuda.synchronize()
    q_idx, n, prefix = oracle.compact(d)
    assert np.array_equal(buf.d_mask.cpu().numpy(), d)
    assert np.array_equal(buf.n_routed.cpu().numpy(), n)
    assert np.array_equal(buf.q_idx.cpu().numpy(), q_idx)
    assert np.array_equal(buf.prefix.cpu().numpy(), prefix)


def test_route_compact_logits_bit_exact():
    B, L = 2, 70001
    z = synth.router_logits(B, L, -1.4, seed=3)
    z[0, :8] = [0.0, -0.0, 1e-30, -1e-30, np.nan, np.inf, -np.inf, -1e-9]
    for thr in (0.0, 0.25):
        d = oracle.route(z, thr)
        p = l2a.params(B, L, L, 2, 1, 64, 8)
        buf = l2a.Buffers.allocate(p, router_dtype=torch.float32)
        buf.router.copy_(torch.from_numpy(z))
        buf.route(l2a.ROUTER_LOGITS_F32, thr)
        torch.cuda.synchronize()
        q_idx, n, prefix = oracle.compact(d)
        assert np.array_equal(buf.d_mask.cpu().numpy(), d)
        assert np.array_equal(buf.q_idx.cpu().numpy(), q_idx)
        assert np.array_equal(buf.n_routed.cpu().numpy(), n)
        assert np.array_equal(buf.prefix.cpu().numpy(), prefix)
    assert list(d[0, :8]) == [0, 0, 0, 0, 0, 1, 0, 0]  # thr = 0.25


def test_route_compact_bf16_logits_bit_exact():
    """bf16 logits are compared in fp32 after an exact upcast: the reference is the fp32 route on the upcast values."""
    B, L = 3, 9001
    z = torch.from_numpy(synth.router_logits(B, L, -0.8416, seed=5)).to(torch.bfloat16)
    z[0, :6] = torch.tensor([0.0, -0.0, float("nan"), float("inf"), -float("inf"), 0.25], dtype=torch.bfloat16)
    z32 = z.float().numpy()
    for thr in (0.0, 0.25):
        d = oracle.route(z32, thr)
        p = l2a.params(B, L, L, 2, 1, 64, 8)
        buf = l2a.Buffers.allocate(p, router_dtype=torch.bfloat16)
        buf.router.copy_(z)
        buf.route(l2a.ROUTER_LOGITS_BF16, thr)
        torch.cuda.synchronize()
        q_idx, n, prefix = oracle.compact(d)
        assert np.array_equal(buf.d_mask.cpu().numpy(), d)
        assert np.array_equal(buf.q_idx.cpu().numpy(), q_idx)
        assert np.array_equal(buf.n_routed.cpu().numpy(), n)
        assert np.array_equal(buf.prefix.cpu().numpy(), prefix)
    assert 0.1 < d.mean() < 0.3
    # the allocation-free entry point takes the same kinds
    buf.d_mask.zero_()
    l2a.l2a_route_compact_static(p, buf.router, l2a.ROUTER_LOGITS_BF16, 0.25, buf.d_mask, buf.q_idx, buf.n_routed,
                                 buf.prefix)
    torch.cuda.synchronize()
    assert np.array_equal(buf.d_mask.cpu().numpy(), d)


# ------------------------------------------------------------------------------- forward, element by element

def test_forward_tiny_config_full():
    """Config 'tiny': B=1, L=1024, one head, D=64, W=128, Bernoulli(0.2), token 0 local-only."""
    cfg = synth.CONFIGS["tiny"]
    d, _ = synth.routing(cfg, synth.seed_for(1))
    c = Case(cfg.B, cfg.L, cfg.Hq, cfg.Hkv, cfg.D, cfg.W, d, synth.seed_for(1), backward=True, scale=1.0 / 8.0)
    c.run_forward()
    c.check_forward_full()


@pytest.mark.parametrize("B,Lq,Lk,Hq,Hkv,D,W,rho", [
    (1, 700, 700, 2, 1, 128, 200, 0.3),      # several tiles, ragged tail, window not a block multiple
    (2, 513, 513, 4, 2, 128, 128, 0.5),      # batch > 1, GQA, one row past a tile boundary
    (1, 300, 1000, 2, 2, 64, 96, 0.4),       # Lk > Lq: bottom-right aligned positions
    (1, 640, 640, 2, 1, 128, 0, 0.2),        # W = 0: local output is v_t
    (1, 600, 600, 1, 1, 64, 5000, 0.2),      # W >= L - 1: local is full causal
    (1, 1, 1, 1, 1, 128, 4, 1.0),            # a single token
    (1, 129, 129, 1, 1, 128, 16, 1.0),       # every token routed, n_c one past a tile
    (1, 1500, 1500, 2, 2, 128, 256, 0.02),   # few routed rows spread over many key blocks
])
def test_forward_matches_oracle(B, Lq, Lk, Hq, Hkv, D, W, rho):
    d = synth.mask_bernoulli(B, Lq, rho, seed=Lq * 7 + W)
    c = Case(B, Lq, Hq, Hkv, D, W, d, seed=Lq + 13 * D + W, Lk=Lk, backward=True)
    c.run_forward()
    c.check_forward_full()


def test_forward_no_routed_rows_and_bit_identity():
    """d == 0 -> O is the sliding-window output; rows with d_t = 0 of a routed run are bit-identical to it."""
    B, L, Hq, Hkv, D, W = 1, 900, 2, 1, 128, 300
    zeros = np.zeros((B, L), np.uint8)
    c0 = Case(B, L, Hq, Hkv, D, W, zeros, seed=5)
    c0.run_forward()
    ref = c0.check_forward_full()
    check_close(to_f64(c0.buf.O), ref["s"], "O == S when nothing is routed")
    d = synth.mask_bernoulli(B, L, 0.3, seed=9)
    c1 = Case(B, L, Hq, Hkv, D, W, d, seed=5)
    c1.run_forward()
    off = torch.from_numpy(~d[0].astype(bool)).cuda()
    assert torch.equal(c1.buf.O[0][off].view(torch.int16), c0.buf.O[0][off].view(torch.int16))


def test_forward_closed_form_zero_keys_long():
    """K == 0 -> uniform soft-max: exact O(L) reference usable at a length where a full oracle run is slow."""
    B, L, Hq, Hkv, D, W = 1, 20000, 2, 1, 128, 4096
    d = synth.mask_bernoulli(B, L, 0.2, seed=1)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=77, backward=True)
    c.buf.K.zero_()
    c.run_forward()
    v = to_f64(c.buf.V)[0, :, 0]
    cs = np.concatenate([np.zeros((1, D)), np.cumsum(v, axis=0)])
    t = np.arange(L)
    lo = np.maximum(0, t - W)
    s_ref = (cs[t + 1] - cs[lo]) / (t - lo + 1)[:, None]
    a_ref = cs[t + 1] / (t + 1)[:, None] * d[0][:, None]
    O = to_f64(c.buf.O)[0]
    for h in range(Hq):
        check_close(O[:, h], s_ref + a_ref, f"O head {h}")
        check_close(to_f64(c.buf.lse_loc)[0, h], np.log(np.minimum(t + 1, W + 1)), "lse_loc", LSE_ABS, LSE_ABS)
    rows = np.nonzero(d[0])[0]
    check_close(to_f64(c.buf.lse_glb)[0, 0, :rows.size], np.log(rows + 1.0), "lse_glb", LSE_ABS, LSE_ABS)


def test_forward_flags_skip_local_and_skip_global():
    B, L, Hq, Hkv, D, W = 1, 520, 2, 1, 128, 64
    d = synth.mask_bernoulli(B, L, 0.4, seed=21)
    ref = None
    for flag in (l2a.FLAG_SKIP_LOCAL, l2a.FLAG_SKIP_GLOBAL):
        c = Case(B, L, Hq, Hkv, D, W, d, seed=31, flags=flag)
        c.run_forward()
        ref = c.oracle_forward() if ref is None else ref
        check_close(to_f64(c.buf.O), ref["a"] if flag == l2a.FLAG_SKIP_LOCAL else ref["s"], f"flag {flag}")


def test_forward_run_twice_is_bit_identical():
    B, L, Hq, Hkv, D, W = 1, 777, 2, 1, 128, 100
    d = synth.mask_bernoulli(B, L, 0.3, seed=2)
    c = Case(B, L, Hq, Hkv, D, W, d, seed=3)
    c.run_forward()
    first = c.buf.O.clone()
    c.run_forward()
    assert torch.equal(first.view(torch.int16), c.buf.O.view(torch.int16))


def test_forward_argument_errors_are_reported_on_the_host():
    p = l2a.params(1, 256, 256, 2, 1, 128, 16)
    buf = l2a.Buffers.allocate(p)
    bad = l2a.params(1, 256, 256, 3, 2, 128, 16)            # Hq % Hkv != 0
    assert l2a.l2a_forward(bad, buf.Q, buf.K, buf.V, buf.d_mask, buf.q_idx, buf.n_routed, buf.prefix, buf.O, None,
                           None, None, None, buf.fwd_ws, check=False) == -1
    d96 = l2a.params(1, 256, 256, 2, 1, 96, 16)             # unsupported head dim
    assert l2a.l2a_forward(d96, buf.Q, buf.K, buf.V, buf.d_mask, buf.q_idx, buf.n_routed, buf.prefix, buf.O, None,
                           None, None, None, buf.fwd_ws, check=False) == -2
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    assert l2a.l2a_forward(p, buf.Q, buf.K, buf.V, buf.d_mask, buf.q_idx, buf.n_routed, buf.prefix, buf.O, None,
                           None, None, None, small, check=False) == -3
    assert l2a.l2a_forward(p, None, buf.K, buf.V, buf.d_mask, buf.q_idx, buf.n_routed, buf.prefix, buf.O, None,
                           None, None, None, buf.fwd_ws, check=False) == -1
    torch.cuda.synchronize()
