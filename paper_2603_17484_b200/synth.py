"""Seeded synthetic inputs for the L2A layer: bf16 Q/K/V/dO tensors and routing decisions.

Holds input generation only -- none of the layer's arithmetic -- so that the CUDA path and the
test oracle can be fed bit-identical inputs.  Tensors are torch CPU bfloat16, layout [B, L, H, D];
``as_u16`` gives the same bits as a numpy uint16 array.

The shapes stand in for Qwen2.5-7B (28 query / 4 KV heads, head dim 128) and Qwen3-8B (32 / 8,
head dim 128) attention; values are i.i.d. N(0, 1) rounded to bf16 (round-to-nearest-even).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

BASE_SEED = 20260317


@dataclass
class Config:
    name: str
    B: int
    L: int
    Hq: int
    Hkv: int
    D: int
    W: int
    routing: str            # "bernoulli" | "logits" | "clustered" | "all" | "none"
    density: float = 0.2
    backward: bool = False
    clear_token0: bool = False
    logit_mean: float = -1.4
    extra: dict = field(default_factory=dict)


# The five workload configurations (routing density of the swept ones is a parameter).
CONFIGS = {
    "tiny": Config("tiny", 1, 1024, 1, 1, 64, 128, "bernoulli", 0.2, False, True),
    "qwen25_7b_32k": Config("qwen25_7b_32k", 1, 32768, 28, 4, 128, 4096, "bernoulli", 0.2),
    "train_64k": Config("train_64k", 1, 65536, 28, 4, 128, 4096, "logits", 0.0808, True),
    "qwen3_8b_128k": Config("qwen3_8b_128k", 1, 131072, 32, 8, 128, 4096, "bernoulli", 0.2),
    "stress_128k": Config("stress_128k", 1, 131072, 32, 8, 128, 4096, "clustered", 0.2, True),
}
CONFIG_INDEX = {"tiny": 1, "qwen25_7b_32k": 2, "train_64k": 3, "qwen3_8b_128k": 4, "stress_128k": 5}


def seed_for(config_index: int, sweep: int = 0) -> int:
    return BASE_SEED + 1000 * config_index + sweep


def normal_bf16(shape, seed: int) -> torch.Tensor:
    """i.i.d. N(0,1) in fp32 from a seeded CPU generator, rounded to bf16."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return torch.randn(shape, generator=g, dtype=torch.float32).to(torch.bfloat16)


def as_u16(t: torch.Tensor) -> np.ndarray:
    """bf16 torch tensor -> numpy uint16 bit patterns (no copy when contiguous)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def qkv(B, L, Hq, Hkv, D, seed: int, with_dO: bool = False, Lk: int | None = None):
    Lk = L if Lk is None else Lk
    out = {
        "Q": normal_bf16((B, L, Hq, D), seed * 4 + 0),
        "K": normal_bf16((B, Lk, Hkv, D), seed * 4 + 1),
        "V": normal_bf16((B, Lk, Hkv, D), seed * 4 + 2),
    }
    if with_dO:
        out["dO"] = normal_bf16((B, L, Hq, D), seed * 4 + 3)
    return out


def mask_bernoulli(B, L, density: float, seed: int, clear_token0: bool = False) -> np.ndarray:
    rng = np.random.default_rng(seed)
    d = (rng.random((B, L)) < density).astype(np.uint8)
    if clear_token0:
        d[:, 0] = 0
    return d


def router_logits(B, L, mean: float, seed: int) -> np.ndarray:
    """fp32 router logits ~ N(mean, 1); the decision is logit >= 0 (sigmoid >= 0.5)."""
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((B, L)) + mean).astype(np.float32)


def mask_clustered(B, L, density: float, seed: int, mean_burst: float = 64.0) -> np.ndarray:
    """Bursts of consecutive routed tokens with geometric length (mean ``mean_burst``).

    Two-state Markov chain over positions: leave a burst with probability 1/mean_burst, enter one
    with probability density / (mean_burst * (1 - density)) so that the stationary routed fraction
    is ``density``; the first state is drawn from the stationary law."""
    d = np.zeros((B, L), np.uint8)
    if density <= 0.0:
        return d
    if density >= 1.0:
        d[:] = 1
        return d
    rng = np.random.default_rng(seed)
    p_leave = 1.0 / mean_burst
    p_enter = density / (mean_burst * (1.0 - density))
    for b in range(B):
        t = 0
        on = rng.random() < density
        while t < L:
            run = int(rng.geometric(p_leave if on else min(1.0, p_enter)))
            if on:
                d[b, t:t + run] = 1
            t += run
            on = not on
    return d


def routing(cfg: Config, seed: int, density: float | None = None):
    """Returns (d uint8 [B, L], logits fp32 [B, L] or None)."""
    rho = cfg.density if density is None else density
    if cfg.routing == "bernoulli":
        return mask_bernoulli(cfg.B, cfg.L, rho, seed, cfg.clear_token0), None
    if cfg.routing == "logits":
        z = router_logits(cfg.B, cfg.L, cfg.logit_mean, seed)
        return (z >= np.float32(0.0)).astype(np.uint8), z
    if cfg.routing == "clustered":
        return mask_clustered(cfg.B, cfg.L, rho, seed), None
    if cfg.routing == "all":
        return np.ones((cfg.B, cfg.L), np.uint8), None
    if cfg.routing == "none":
        return np.zeros((cfg.B, cfg.L), np.uint8), None
    raise ValueError(cfg.routing)


def pairs_local(L: int, W: int) -> int:
    """(query, key) pairs inside the causal sliding window: sum_t min(t, W) + 1."""
    if L <= W:
        return L * (L + 1) // 2
    return W * (W + 1) // 2 + (W + 1) * (L - W)


def pairs_global(d_row: np.ndarray) -> int:
    """Causal pairs of routed rows: sum over routed t of (t + 1)."""
    t = np.nonzero(d_row)[0].astype(np.int64)
    return int((t + 1).sum())


def useful_flops(cfg: Config, d: np.ndarray, backward: bool) -> tuple[float, float]:
    """(forward, backward) useful FLOPs: 4*D per pair per query head forward (two GEMMs), 10*D
    backward (five GEMMs); only in-window local pairs and causal pairs of routed rows count."""
    pairs = sum(pairs_local(cfg.L, cfg.W) + pairs_global(d[b]) for b in range(cfg.B))
    fwd = 4.0 * cfg.D * cfg.Hq * pairs
    bwd = 10.0 * cfg.D * cfg.Hq * pairs if backward else 0.0
    return fwd, bwd
