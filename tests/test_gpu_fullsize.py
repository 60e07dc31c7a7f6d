"""GPU parity at the benchmark sizes, in the launch configuration bench.py times: outputs the oracle can
compute one by one (>= 4096 sampled rows per head for O / dQ, sampled key positions for dK / dV) plus
identities that hold at any size.  The oracle work is sized for a few minutes on ~16 host cores."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import check_close, check_same_or_rounding, to_f64, LSE_ABS

pytestmark = pytest.mark.gpu

ROWS_PER_HEAD = 4096

# The two launch configurations of a test read the same seeded inputs, so the oracle's answer is computed once.
_ORACLE = {}


def once(key, fn):
    if key not in _ORACLE:
        _ORACLE[key] = fn()
    return _ORACLE[key]


def sample_rows(d_row: np.ndarray, n: int, seed: int) -> np.ndarray:
    """n distinct rows: at least a quarter routed (when there are enough), first and last tile always hit."""
    rng = np.random.default_rng(seed)
    L = d_row.size
    routed = np.nonzero(d_row)[0]
    fixed = np.array([0, 1, 127, 128, L - 129, L - 128, L - 1])
    take_r = min(routed.size, n // 4)
    pick_r = rng.choice(routed, take_r, replace=False) if take_r else np.empty(0, np.int64)
    rest = np.setdiff1d(np.arange(L), np.concatenate([fixed, pick_r]))
    pick = rng.choice(rest, n - take_r - fixed.size, replace=False)
    return np.sort(np.concatenate([fixed, pick_r, pick])).astype(np.int32)


# both launch configurations bench.py can time: plain, and with the shared-projection fusion
SHARED = pytest.mark.parametrize("shared", [False, True], ids=["plain", "shared_window"])


def setup(name, rho=None, backward=False, sweep=0, shared=False, **override):
    """override: fields of the named configuration to replace (routing, logit_mean, ...)."""
    cfg = synth.CONFIGS[name]
    if override:
        cfg = synth.Config(**{**cfg.__dict__, **override})
    seed = synth.seed_for(synth.CONFIG_INDEX[name], sweep)
    d, logits = synth.routing(cfg, seed, density=rho)
    host = synth.qkv(cfg.B, cfg.L, cfg.Hq, cfg.Hkv, cfg.D, seed, with_dO=backward)
    p = l2a.params(cfg.B, cfg.L, cfg.L, cfg.Hq, cfg.Hkv, cfg.D, cfg.W,
                   flags=(l2a.FLAG_SAVE_FOR_BWD if backward else 0) | (l2a.FLAG_SHARED_WINDOW if shared else 0))
    buf = l2a.Buffers.allocate(p, backward=backward, router_dtype=torch.float32 if logits is not None else torch.uint8)
    if shared and not backward:
        buf.lse_loc = torch.empty((cfg.B, cfg.Hq, cfg.L), dtype=torch.float32, device="cuda")
    for k in ("Q", "K", "V") + (("dO",) if backward else ()):
        getattr(buf, k).copy_(host[k])
    buf.router.copy_(torch.from_numpy(logits if logits is not None else d))
    buf.O.fill_(float("nan"))
    buf.route(l2a.ROUTER_LOGITS_F32 if logits is not None else l2a.ROUTER_MASK_U8, 0.0)
    buf.forward()
    if backward:
        buf.backward()
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(buf.fwd_ws) == 0
    if backward:
        assert l2a.l2a_workspace_status(buf.bwd_ws) == 0
    sh = oracle.Shape(cfg.B, cfg.L, cfg.L, cfg.Hq, cfg.Hkv, cfg.D, cfg.W)
    u16 = {k: synth.as_u16(v) for k, v in host.items()}
    q_idx, n, prefix = oracle.compact(d)
    assert np.array_equal(buf.q_idx.cpu().numpy(), q_idx)
    assert np.array_equal(buf.n_routed.cpu().numpy(), n)
    assert np.array_equal(buf.prefix.cpu().numpy(), prefix)
    assert np.array_equal(buf.d_mask.cpu().numpy(), d)
    return cfg, d, buf, sh, u16


def rows_for_all_heads(cfg, d, seed):
    rt = sample_rows(d[0], ROWS_PER_HEAD, seed)
    rh = np.repeat(np.arange(cfg.Hq, dtype=np.int32), rt.size)
    rt_all = np.tile(rt, cfg.Hq)
    return np.zeros_like(rt_all), rh, rt_all, rt


@SHARED
def test_forward_128k_sampled_rows(shared):
    """Qwen3-8B-shaped 128K prefill forward, Bernoulli(0.2): 4096 sampled rows of every head."""
    cfg, d, buf, sh, u16 = setup("qwen3_8b_128k", rho=0.2, sweep=2, shared=shared)
    rb, rh, rt, rows = rows_for_all_heads(cfg, d, seed=41)
    ref = once("fwd128k", lambda: oracle.forward_rows(sh, u16["Q"], u16["K"], u16["V"], d, rb, rh, rt))
    idx = torch.from_numpy(rows.astype(np.int64)).cuda()
    got = to_f64(buf.O[0].index_select(0, idx))                      # [rows, Hq, D]
    want = ref["o"].reshape(cfg.Hq, rows.size, cfg.D).transpose(1, 0, 2)
    check_close(got, want, "O (sampled rows, 128K)")
    assert torch.isfinite(buf.O.float()).all()


@SHARED
def test_forward_32k_sampled_rows(shared):
    """Qwen2.5-7B-shaped 32K forward (28 query / 4 KV heads), Bernoulli(0.2)."""
    cfg, d, buf, sh, u16 = setup("qwen25_7b_32k", shared=shared)
    rb, rh, rt, rows = rows_for_all_heads(cfg, d, seed=42)
    ref = once("fwd32k", lambda: oracle.forward_rows(sh, u16["Q"], u16["K"], u16["V"], d, rb, rh, rt))
    idx = torch.from_numpy(rows.astype(np.int64)).cuda()
    got = to_f64(buf.O[0].index_select(0, idx))
    want = ref["o"].reshape(cfg.Hq, rows.size, cfg.D).transpose(1, 0, 2)
    check_close(got, want, "O (sampled rows, 32K)")


@SHARED
def test_train_64k_forward_backward_sampled(shared):
    """Training-step shape: L=65536, 28/4 heads, router logits ~ N(-1.4, 1) thresholded at 0 (about 8 % routed)."""
    cfg, d, buf, sh, u16 = setup("train_64k", backward=True, shared=shared)
    assert 0.07 < d.mean() < 0.09
    rb, rh, rt, rows = rows_for_all_heads(cfg, d, seed=43)
    idx = torch.from_numpy(rows.astype(np.int64)).cuda()
    # dQ of the sampled rows, every head
    want = once("dq64k", lambda: oracle.dq_rows(sh, u16["Q"], u16["K"], u16["V"], d, u16["dO"], rb, rh, rt))
    got = to_f64(buf.dQ[0].index_select(0, idx))
    check_close(got, want.reshape(cfg.Hq, rows.size, cfg.D).transpose(1, 0, 2), "dQ (sampled rows, 64K)")
    # saved statistics on a subset (they feed the backward)
    sub = slice(0, rows.size, 16)
    ref = once("stat64k", lambda: oracle.forward_rows(sh, u16["Q"], u16["K"], u16["V"], d, np.zeros_like(rows[sub]),
                                                      np.full_like(rows[sub], 5), rows[sub]))
    check_close(to_f64(buf.lse_loc[0, 5].index_select(0, idx[sub])), ref["lse_loc"], "lse_loc", LSE_ABS, LSE_ABS)
    # dK / dV at sampled key positions of one KV group: late keys, mid-sequence keys, early keys
    L = cfg.L
    js = np.array([L - 1, L - 2, L - 100, L - 129, L - 700, L - 1000, L // 2, L // 2 + 77, 300, 5], np.int32)
    g = 2
    dk, dv = once("dkv64k", lambda: oracle.dkv_cols(sh, u16["Q"], u16["K"], u16["V"], d, u16["dO"], 0, g, js))
    jt = torch.from_numpy(js.astype(np.int64)).cuda()
    check_close(to_f64(buf.dK[0].index_select(0, jt)[:, g]), dk, "dK (sampled keys, 64K)")
    check_close(to_f64(buf.dV[0].index_select(0, jt)[:, g]), dv, "dV (sampled keys, 64K)")


@SHARED
def test_stress_128k_backward_identities_and_rows(shared):
    """The benchmark's own workload (128K, clustered routing rho = 0.2, fwd + bwd): 4096 sampled dQ rows of every
    head, the dV column-sum identity, and finiteness of every output."""
    cfg, d, buf, sh, u16 = setup("stress_128k", rho=0.2, backward=True, sweep=2, shared=shared)
    for t in (buf.O, buf.dQ, buf.dK, buf.dV):
        assert torch.isfinite(t.float()).all()
    rows = sample_rows(d[0], ROWS_PER_HEAD, seed=44)
    rh = np.repeat(np.arange(cfg.Hq, dtype=np.int32), rows.size)
    rt = np.tile(rows, cfg.Hq)
    want = once("dq128k", lambda: oracle.dq_rows(sh, u16["Q"], u16["K"], u16["V"], d, u16["dO"], np.zeros_like(rt), rh, rt))
    idx = torch.from_numpy(rows.astype(np.int64)).cuda()
    check_close(to_f64(buf.dQ[0].index_select(0, idx)), want.reshape(cfg.Hq, rows.size, cfg.D).transpose(1, 0, 2),
                "dQ (sampled rows, 128K)")
    # sum_j dV_j = sum_t (1 + d_t) dO_t per KV group (each soft-max row sums to one); fp32 sums on the GPU
    w = torch.from_numpy((1 + d[0]).astype(np.float32)).cuda()
    G = cfg.Hq // cfg.Hkv
    want_sum = (buf.dO[0].float() * w[:, None, None]).view(cfg.L, cfg.Hkv, G, cfg.D).sum(dim=(0, 2)).double()
    got_sum = buf.dV[0].double().sum(dim=0)
    # every dV entry carries a bf16 rounding of relative size 2^-9; they add up like a random walk
    scale = buf.dV[0].float().abs().mean().item() * 2.0 ** -9 * np.sqrt(cfg.L) * 8 + 1.0
    assert (got_sum - want_sum).abs().max().item() <= scale, ((got_sum - want_sum).abs().max().item(), scale)


def test_stress_128k_shared_window_agrees_with_independent_modules_everywhere():
    """Every element of O, dQ, dK, dV of the benchmark workload, computed with and without the shared-window fusion:
    two bf16 results of the same quantity, each within the bound of the exact value, so within twice the bound of
    each other (the sampled-row tests above tie both to the oracle; this one covers every tile of the launch)."""
    outs = []
    for shared in (False, True):
        cfg, d, buf, sh, u16 = setup("stress_128k", rho=0.2, backward=True, sweep=2, shared=shared)
        outs.append({k: getattr(buf, k).float() for k in ("O", "dQ", "dK", "dV")})
        del buf
        torch.cuda.empty_cache()
    for k in ("O", "dQ", "dK", "dV"):
        a, b = outs[0][k], outs[1][k]
        err = (a - b).abs()
        bound = 2 * (2e-2 + 2.0 ** -8 * a.abs())
        n_over = int((err > bound).sum().item())
        assert n_over <= max(1, int(1e-5 * err.numel())), (k, n_over, err.max().item())
        assert err.mean().item() <= 2 * (2e-3 + 2.0 ** -9 * a.abs().mean().item()), (k, err.mean().item())


@SHARED
def test_forward_128k_constant_values_every_row(shared):
    """V = c for every key (one vector per KV head): every soft-max average is c, so o_t = (1 + d_t) c for every row
    of the 128K launch, whatever the scores are -- a check of every tile, mask edge and scatter of the forward."""
    cfg = synth.CONFIGS["stress_128k"]
    seed = synth.seed_for(synth.CONFIG_INDEX["stress_128k"], 3)
    d, _ = synth.routing(cfg, seed, density=0.2)
    p = l2a.params(cfg.B, cfg.L, cfg.L, cfg.Hq, cfg.Hkv, cfg.D, cfg.W,
                   flags=l2a.FLAG_SAVE_FOR_BWD | (l2a.FLAG_SHARED_WINDOW if shared else 0))
    buf = l2a.Buffers.allocate(p, backward=True)
    g = torch.Generator(device="cuda").manual_seed(seed)
    buf.Q.copy_(torch.randn(buf.Q.shape, generator=g, device="cuda"))
    buf.K.copy_(torch.randn(buf.K.shape, generator=g, device="cuda"))
    c = torch.randn((cfg.Hkv, cfg.D), generator=g, device="cuda").to(torch.bfloat16)
    buf.V.copy_(c.expand(cfg.B, cfg.L, cfg.Hkv, cfg.D))
    buf.router.copy_(torch.from_numpy(d))
    buf.O.fill_(float("nan"))
    buf.route()
    buf.forward()
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(buf.fwd_ws) == 0
    G = cfg.Hq // cfg.Hkv
    want = c.float().repeat_interleave(G, dim=0)[None, None] * (1.0 + buf.d_mask.float())[:, :, None, None]
    err = (buf.O.float() - want).abs()
    bound = 2e-2 + 2.0 ** -8 * want.abs()
    assert torch.isfinite(buf.O.float()).all()
    assert int((err > bound).sum().item()) == 0, err.max().item()
    assert err.mean().item() <= 2e-3 + 2.0 ** -9 * want.abs().mean().item()


@SHARED
def test_stress_128k_backward_is_reproducible_and_linear_in_dO(shared):
    """dK and dV are accumulated on chip in a fixed order: a second run gives the same bits in every element of the 128K
    launch, and doubling dO (exact in bf16 and fp32) doubles every element exactly.  dQ is summed over the key blocks
    with atomic fp32 additions: the same up to the rounding of sums taken in another order.  Races or stale tiles
    anywhere in the launch would show up here."""
    cfg, d, buf, sh, u16 = setup("stress_128k", rho=0.2, backward=True, sweep=2, shared=shared)
    first = {k: getattr(buf, k).clone() for k in ("dQ", "dK", "dV")}
    for k in first:
        getattr(buf, k).fill_(float("nan"))
    buf.backward()
    torch.cuda.synchronize()
    for k in ("dK", "dV"):
        assert torch.equal(getattr(buf, k).view(torch.int16), first[k].view(torch.int16)), k
    check_same_or_rounding(first["dQ"], buf.dQ, "dQ, second run")
    buf.dO.mul_(2.0)
    buf.backward()
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(buf.bwd_ws) == 0
    for k in ("dK", "dV"):
        assert torch.equal(getattr(buf, k).float(), 2.0 * first[k].float()), k
    check_same_or_rounding((2.0 * first["dQ"].float()).to(torch.bfloat16), buf.dQ, "dQ, doubled dO")
