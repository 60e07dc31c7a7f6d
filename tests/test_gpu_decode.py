"""Decode step against the oracle: the layer with a single query row placed at the end of the cache."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_17484_b200 import l2a, synth
from tests.gpu_util import check_close, to_f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,Lk,Hq,Hkv,D,W", [
    (3, 1, 2, 1, 128, 16),          # cache of one token
    (4, 700, 4, 1, 128, 200),       # G = 4
    (2, 5000, 28, 4, 128, 4096),    # Qwen2.5-7B heads (G = 7), window larger than most of the cache
    (3, 9001, 32, 8, 128, 4096),    # Qwen3-8B heads
    (2, 3000, 4, 4, 64, 100),       # head dim 64, no grouping
])
def test_decode_matches_oracle(B, Lk, Hq, Hkv, D, W):
    t = synth.qkv(B, 1, Hq, Hkv, D, seed=Lk + Hq, Lk=Lk)
    d = (np.arange(B) % 2).astype(np.uint8)[:, None]          # alternate routed / not routed, shape [B, 1]
    p = l2a.params(B, 1, Lk, Hq, Hkv, D, W)
    ws = torch.empty(l2a.l2a_decode_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    q, K, V = (t[k].cuda() for k in ("Q", "K", "V"))
    O = torch.full((B, 1, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    l2a.l2a_decode(p, q, K, V, torch.from_numpy(d[:, 0].copy()).cuda(), O, ws)
    torch.cuda.synchronize()
    sh = oracle.Shape(B, 1, Lk, Hq, Hkv, D, W)
    ref = oracle.forward_full(sh, synth.as_u16(t["Q"]), synth.as_u16(t["K"]), synth.as_u16(t["V"]), d)
    check_close(to_f64(O), ref["o"], "decode O")
    # a not-routed token equals the sliding-window output exactly as computed for d == 0
    O0 = torch.empty_like(O)
    l2a.l2a_decode(p, q, K, V, None, O0, ws)
    torch.cuda.synchronize()
    check_close(to_f64(O0), ref["s"], "decode O with no routing (local only)")


@pytest.mark.parametrize("B,Lk,pos,Hq,Hkv,D,W", [
    (2, 4096, 3000, 8, 2, 128, 512),     # cache allocated ahead of the sequence
    (1, 70000, 69990, 32, 8, 128, 4096), # one sequence: the chunk plan shrinks its chunks to fill the SMs
    (2, 1000, 63, 4, 2, 64, 31),         # position on a tile boundary, window smaller than a tile
])
def test_decode_ignores_cache_past_the_position(B, Lk, pos, Hq, Hkv, D, W):
    """Rows of the cache after the new token's position are not part of the sequence yet: whatever they hold (NaN
    here) must not reach the output."""
    t = synth.qkv(B, 1, Hq, Hkv, D, seed=pos, Lk=Lk)
    d = np.ones((B, 1), dtype=np.uint8)
    p = l2a.params(B, 1, Lk, Hq, Hkv, D, W, q_pos_offset=pos)
    ws = torch.empty(l2a.l2a_decode_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    q, K, V = (t[k].cuda() for k in ("Q", "K", "V"))
    K[:, pos + 1:] = float("nan")
    V[:, pos + 1:] = float("nan")
    O = torch.full((B, 1, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    l2a.l2a_decode(p, q, K, V, torch.from_numpy(d[:, 0].copy()).cuda(), O, ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(ws) == 0
    sh = oracle.Shape(B, 1, Lk, Hq, Hkv, D, W, q_pos_offset=pos)
    ref = oracle.forward_full(sh, synth.as_u16(t["Q"]), synth.as_u16(t["K"]), synth.as_u16(t["V"]), d)
    check_close(to_f64(O), ref["o"], "decode O, position before the end of the cache")


def test_decode_pruned_layer_ring_cache():
    """A layer whose Global Attention was pruned (Section 3.4, sparsity-based layer pruning) keeps only the last
    W + 1 keys.  Attention does not depend on the order of the keys, so the cache can be a ring buffer: the decode
    call with d = NULL over the W + 1 slots, in whatever rotation they are, gives the sliding-window output."""
    B, L, Hq, Hkv, D, W = 2, 3000, 8, 2, 128, 511
    t = synth.qkv(B, 1, Hq, Hkv, D, seed=99, Lk=L)
    sh = oracle.Shape(B, 1, L, Hq, Hkv, D, W)
    ref = oracle.forward_full(sh, synth.as_u16(t["Q"]), synth.as_u16(t["K"]), synth.as_u16(t["V"]),
                              np.zeros((B, 1), dtype=np.uint8))
    # ring buffer of W + 1 slots: position j lives in slot j % (W + 1)
    slots = W + 1
    order = torch.tensor([(L - slots + i) for i in range(slots)])
    ring = torch.empty(slots, dtype=torch.long)
    ring[order % slots] = order
    Kr, Vr = t["K"][:, ring].contiguous().cuda(), t["V"][:, ring].contiguous().cuda()
    p = l2a.params(B, 1, slots, Hq, Hkv, D, W)
    ws = torch.empty(l2a.l2a_decode_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    O = torch.empty((B, 1, Hq, D), dtype=torch.bfloat16, device="cuda")
    l2a.l2a_decode(p, t["Q"].cuda(), Kr, Vr, None, O, ws)
    torch.cuda.synchronize()
    check_close(to_f64(O), ref["s"], "decode over a ring-buffer local cache")


def test_decode_full_size_cache():
    """The benchmark's decode configuration (128K-token cache, 32/8 heads, 2048-key chunks): a decode step is a
    single query row per sequence, so the oracle computes every output element."""
    cfg = synth.CONFIGS["qwen3_8b_128k"]
    B, Lk = 2, cfg.L
    t = synth.qkv(B, 1, cfg.Hq, cfg.Hkv, cfg.D, seed=2024, Lk=Lk)
    d = np.array([[1], [0]], dtype=np.uint8)
    p = l2a.params(B, 1, Lk, cfg.Hq, cfg.Hkv, cfg.D, cfg.W)
    ws = torch.empty(l2a.l2a_decode_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    O = torch.full((B, 1, cfg.Hq, cfg.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    l2a.l2a_decode(p, t["Q"].cuda(), t["K"].cuda(), t["V"].cuda(), torch.from_numpy(d[:, 0].copy()).cuda(), O, ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(ws) == 0
    sh = oracle.Shape(B, 1, Lk, cfg.Hq, cfg.Hkv, cfg.D, cfg.W)
    ref = oracle.forward_full(sh, synth.as_u16(t["Q"]), synth.as_u16(t["K"]), synth.as_u16(t["V"]), d)
    check_close(to_f64(O), ref["o"], "decode O at 128K")


def _decode_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        B = int(rng.integers(1, 5))
        Lk = int(rng.choice([1, 2, 63, 64, 65, 129, 1000, 2049, 4097, 6000]))
        pos = Lk - 1 - int(rng.choice([0, 0, 0, 1, 17])) if Lk > 20 else Lk - 1
        Hkv = int(rng.integers(1, 3))
        G = int(rng.integers(1, 9))
        D = int(rng.choice([64, 128]))
        W = int(rng.choice([0, 1, 63, 64, 500, 4096]))
        out.append((B, Lk, pos, Hkv * G, Hkv, D, W, 500 + i))
    return out


@pytest.mark.parametrize("B,Lk,pos,Hq,Hkv,D,W,seed", _decode_shapes(16, 20260317))
def test_decode_random_shape(B, Lk, pos, Hq, Hkv, D, W, seed):
    t = synth.qkv(B, 1, Hq, Hkv, D, seed=seed, Lk=Lk)
    d = (np.random.default_rng(seed).random((B, 1)) < 0.5).astype(np.uint8)
    p = l2a.params(B, 1, Lk, Hq, Hkv, D, W, q_pos_offset=pos)
    ws = torch.empty(l2a.l2a_decode_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    O = torch.full((B, 1, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    l2a.l2a_decode(p, t["Q"].cuda(), t["K"].cuda(), t["V"].cuda(), torch.from_numpy(d[:, 0].copy()).cuda(), O, ws)
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(ws) == 0
    sh = oracle.Shape(B, 1, Lk, Hq, Hkv, D, W, q_pos_offset=pos)
    ref = oracle.forward_full(sh, synth.as_u16(t["Q"]), synth.as_u16(t["K"]), synth.as_u16(t["V"]), d)
    check_close(to_f64(O), ref["o"], "decode O")
