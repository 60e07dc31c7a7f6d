#!/usr/bin/env python
"""Benchmark of the L2A hot path on B200: one step = route/compact + forward + backward of one layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--density RHO] [--impl reference]

Prints ONE JSON line (rank 0).  ``value`` is useful TFLOP/s with inputs resident in HBM, the two modules run
independently (each on the Q/K/V it is given -- the benchmark passes the same set to both); ``e2e`` is the same metric
through the host-buffer C-ABI calls with every step's transfers inside the timed region (two steps in flight on
alternating device tensors, l2a_step_host_async; ``e2e.blocking_step_ms`` is one synchronous l2a_step_host call); ``roofline`` describes the dominant kernel
(timed with CUDA events at the phase boundaries the library records on its own stream; ``achieved`` counts the useful
pairs of the metric, ``achieved_visited`` the pairs the launch really processes; ``traffic`` scales the DRAM bytes of
the ncu capture of the same kernel on the 32K case); ``cpu_baseline`` times the fp64 oracle on a bounded sample of the
workload at its full length and extrapolates the layer.  On the default workload three labelled secondary figures
follow: ``shared_window_fusion`` (valid only because one Q/K/V set feeds both modules here), ``density_0.5`` and
``dense_reference`` (every token routed: the build's own dense path).  With N > 1 every rank runs an independent replica
of the workload (the path has no exchange step).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_17484_b200 import replicas, synth  # noqa: E402

METRIC = "L2A fwd+bwd useful TFLOP/s at 128K (one layer, one GPU)"
KERNELS_PER_STEP = 11  # route: count, scan | fwd: gather, local, global | bwd: gather x2, delta, zero, five-GEMM kernel, merge
FWD_PHASES = ("gather_q", "attn_fwd_local", "attn_fwd_global")
BWD_PHASES = ("gather_q_dO", "bwd_delta_zero", "bwd", "bwd_dq_merge")
# DRAM read + write over algorithmic bytes of a launch, from the ncu captures of the 32K case (profiles/)
TRAFFIC_RATIO = {"bwd": 1.15, "attn_fwd_local": 0.94, "attn_fwd_global": 1.17}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            m = json.load(f)
        return {"burst": m["bf16_tflops"], "sustained": m.get("bf16_tflops_sustained", m["bf16_tflops"]),
                "hbm_gbs": m["hbm_gbs"], "source": "measured"}
    return {"burst": 1590.0, "sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="l2a_clocks_", suffix=".csv")
            self.out = os.fdopen(fd, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, smax, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        with open(self.path) as f:
            for line in f:
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1])); smax.append(float(parts[2])); power.append(float(parts[3]))
                except ValueError:
                    continue
                for n, v in zip(names, parts[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "power_w_max": float(max(power)), "samples": len(sm)}


def make_workload(args, seed_offset=0):
    cfg = synth.CONFIGS[args.workload]
    idx = synth.CONFIG_INDEX[args.workload]
    rho = cfg.density if args.density is None else args.density
    seed = synth.seed_for(idx, int(round(rho * 10))) + replicas.rank_seed_offset(seed_offset)
    if args.routing:
        cfg = synth.Config(**{**cfg.__dict__, "routing": args.routing})
    if getattr(args, "kv_heads", None):       # a slice of the workload: the first KV heads and their query heads
        cfg = synth.Config(**{**cfg.__dict__, "Hkv": args.kv_heads, "Hq": args.kv_heads * (cfg.Hq // cfg.Hkv)})
    d, logits = synth.routing(cfg, seed, density=rho)
    return cfg, rho, seed, d, logits


def issued_tile_pairs(mask, L, W, shared=False, tile=128):
    """Score elements the tensor cores really compute, (local, global): every (128-row tile, 128-key block) pair a launch
    issues MMAs for counts whole (edge blocks are masked after the product, ragged tiles are padded with zero rows).
    Local: the blocks between the first row's window start and the last row's diagonal; global: the blocks up to the
    last row of each compact tile of 128 routed rows (up to its position - W - 1 with the shared-window flag)."""
    T = tile
    loc = glb = 0
    for b in range(mask.shape[0]):
        r0 = np.arange(0, L, T, dtype=np.int64)
        r1 = np.minimum(r0 + T, L) - 1
        loc += int((r1 // T - np.maximum(r0 - W, 0) // T + 1).sum())
        t = np.nonzero(mask[b])[0].astype(np.int64)
        if len(t):
            last = t[np.minimum(np.arange(T - 1, len(t) + T - 1, T), len(t) - 1)]      # last row of each compact tile
            bound = last - (W + 1 if shared else 0)
            glb += int((bound[bound >= 0] // T + 1).sum())
    return loc * T * T, glb * T * T


def cpu_oracle_sample(cfg, seed, d, rows_per_head=96, key_span=2500, n_keys=8, backward=True, host=None):
    """The fp64 oracle on a bounded sample of the workload at its FULL length: `rows_per_head` random rows of the second
    half of the sequence (half of them routed when there are enough) in every head -- forward (s, a, o) and dQ -- and
    dK / dV at `n_keys` key positions of the last `key_span` tokens of one KV group.  Returns the pairs per second of
    each leg and the whole layer's time extrapolated from them (labelled as such by the caller)."""
    import oracle
    L = cfg.L
    t = host if host is not None else synth.qkv(cfg.B, L, cfg.Hq, cfg.Hkv, cfg.D, seed, with_dO=True)
    Q, K, V = (synth.as_u16(t[k]) for k in ("Q", "K", "V"))
    dO = synth.as_u16(t["dO"]) if backward else None
    sh = oracle.Shape(cfg.B, L, L, cfg.Hq, cfg.Hkv, cfg.D, cfg.W)
    rng = np.random.default_rng(seed)
    routed = np.nonzero(d[0][L // 2:])[0] + L // 2
    plain = np.nonzero(d[0][L // 2:] == 0)[0] + L // 2
    n_r = min(routed.size, rows_per_head // 2)
    n_p = min(plain.size, rows_per_head - n_r)
    rows = np.sort(np.concatenate([rng.choice(routed, n_r, replace=False) if n_r else np.empty(0, np.int64),
                                   rng.choice(plain, n_p, replace=False) if n_p else np.empty(0, np.int64)])).astype(np.int32)
    rh = np.repeat(np.arange(cfg.Hq, dtype=np.int32), rows.size)
    rt = np.tile(rows, cfg.Hq)
    rb = np.zeros_like(rt)
    pairs_rows = int(sum(min(int(r), cfg.W) + 1 + (int(r) + 1 if d[0][r] else 0) for r in rows)) * cfg.Hq
    cores = oracle.num_threads()  # builds/loads outside the timed region
    t0 = time.perf_counter()
    oracle.forward_rows(sh, Q, K, V, d, rb, rh, rt)
    t_fwd = time.perf_counter() - t0
    out = {"cores": cores, "pairs_rows": pairs_rows, "fwd_pairs_per_s": pairs_rows / t_fwd, "seconds": t_fwd}
    if backward:
        t0 = time.perf_counter()
        oracle.dq_rows(sh, Q, K, V, d, dO, rb, rh, rt)
        t_dq = time.perf_counter() - t0
        js = np.sort(rng.choice(np.arange(L - key_span, L), n_keys, replace=False)).astype(np.int32)
        G = cfg.Hq // cfg.Hkv
        # pairs the key-sampled mode has to visit: whole rows of every query that sees one of the keys
        jmin = int(js.min())
        vis = 0
        for r in range(jmin, L):
            if any(r - cfg.W <= j <= r for j in js):
                vis += min(r, cfg.W) + 1
            if d[0][r] and jmin <= r:
                vis += r + 1
        vis *= G
        t0 = time.perf_counter()
        oracle.dkv_cols(sh, Q, K, V, d, dO, 0, cfg.Hkv - 1, js)
        t_dkv = time.perf_counter() - t0
        out.update(dq_pairs_per_s=pairs_rows / t_dq, dkv_pairs_per_s=vis / t_dkv, pairs_keys=vis,
                   seconds=t_fwd + t_dq + t_dkv)
    return out


def cpu_extrapolate(cfg, d, sample, backward):
    """Whole-layer oracle time from the measured pairs per second (an extrapolation, never a measurement)."""
    pairs = sum(synth.pairs_local(cfg.L, cfg.W) + synth.pairs_global(d[b]) for b in range(cfg.B)) * cfg.Hq
    secs = pairs / sample["fwd_pairs_per_s"]
    if backward:
        secs += pairs / sample["dq_pairs_per_s"] + pairs / sample["dkv_pairs_per_s"]
    flops = (4.0 + (10.0 if backward else 0.0)) * cfg.D * pairs
    return flops / secs / 1e12, secs


CPU_SAMPLE_TEXT = ("fp64 oracle at the workload's full length on a bounded sample: {rows} random rows of the second half "
                   "of the sequence in each of the {heads} heads (forward outputs and dQ; {pr:.3g} pairs) and dK/dV at "
                   "{keys} key positions of the last {span} tokens of one KV group ({pk:.3g} pairs), {secs:.1f} s in "
                   "all; value = the layer's useful FLOPs / the whole-layer time EXTRAPOLATED from the measured pairs "
                   "per second of each leg ({ext:.0f} s)")


def run_reference(args):
    """Reference arm: the fp64 oracle as it stands on the host cores, a bounded sample of the same workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, rho, seed, d, _ = make_workload(args)
    host = synth.qkv(cfg.B, cfg.L, cfg.Hq, cfg.Hkv, cfg.D, seed, with_dO=True)
    kw = dict(rows_per_head=args.ref_rows, key_span=1000, n_keys=4, host=host)
    for _ in range(args.warmup):
        cpu_oracle_sample(cfg, seed, d, **{**kw, "rows_per_head": 2, "key_span": 200, "n_keys": 1})
    t0 = time.perf_counter()
    samples = [cpu_oracle_sample(cfg, seed + i, d, **kw) for i in range(args.steps)]
    total = time.perf_counter() - t0
    vals = [cpu_extrapolate(cfg, d, sm, True) for sm in samples]
    value = float(np.mean([v[0] for v in vals]))
    sm = samples[0]
    sample = CPU_SAMPLE_TEXT.format(rows=args.ref_rows, heads=cfg.Hq, pr=sm["pairs_rows"], keys=4, span=1000,
                                    pk=sm["pairs_keys"], secs=sm["seconds"], ext=vals[0][1])
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / max(1, args.steps) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "B": cfg.B, "L": cfg.L, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
                   "W": cfg.W, "routing": args.routing or cfg.routing, "density": float(d.mean()), "pass": "fwd+bwd",
                   "sampled": True},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": sm["cores"], "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_decode(args):
    """Decode-step measurement (not the headline metric): one new token per sequence against a 128K-token cache,
    local window always, whole cache for the routed sequences.  HBM roofline."""
    from paper_2603_17484_b200 import l2a
    torch.cuda.set_device(0)
    cfg = synth.CONFIGS["qwen3_8b_128k"]
    B, Lk = args.decode_batch, cfg.L
    rho = 0.2 if args.density is None else args.density
    p = l2a.params(B, 1, Lk, cfg.Hq, cfg.Hkv, cfg.D, cfg.W)
    g = torch.Generator(device="cuda"); g.manual_seed(7)
    q = torch.randn((B, 1, cfg.Hq, cfg.D), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    K = torch.randn((B, Lk, cfg.Hkv, cfg.D), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    V = torch.randn((B, Lk, cfg.Hkv, cfg.D), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    d_host = (np.random.default_rng(11).random(B) < rho).astype(np.uint8)
    d = torch.from_numpy(d_host).cuda()
    O = torch.empty((B, 1, cfg.Hq, cfg.D), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(l2a.l2a_decode_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    for _ in range(max(3, args.warmup)):
        l2a.l2a_decode(p, q, K, V, d, O, ws)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        l2a.l2a_decode(p, q, K, V, d, O, ws)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    row = cfg.Hkv * cfg.D * 2 * 2                                   # K and V bytes of one cached position
    alg_bytes = float(B * (cfg.W + 1) * row + int(d_host.sum()) * Lk * row)
    peaks = measured_peaks()
    gbs = alg_bytes / ms / 1e6
    print(json.dumps({
        "metric": "L2A decode step, achieved HBM GB/s", "value": gbs, "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "decode_128k", "B": B, "Lk": Lk, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D, "W": cfg.W,
                   "routed_sequences": int(d_host.sum()),
                   "l2_policy": "K/V cache of %.1f GB exceeds L2" % (2 * K.numel() * 2 / 1e9)},
        "roofline": {"bound": "hbm", "kernel": "decode_split_kernel", "achieved": gbs, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                     # ncu capture of a 4-sequence case: DRAM read + write = 0.9975 x algorithmic bytes; scaled
                     "traffic": 0.9975 * alg_bytes, "traffic_source": "scaled from the 4-sequence ncu capture",
                     "algorithmic_bytes_per_launch": alg_bytes},
        "gpu_launches": 2 * args.steps}), flush=True)


def run_router(args):
    """Router kernels on the headline shape (not the headline metric): logits from the local output (Eq. 3) and
    the backward of Eq. 7 with dS_loc = dO + dz w.  HBM roofline; S, dO and dS_loc are 1.07 GB each (exceed L2)."""
    from paper_2603_17484_b200 import l2a
    torch.cuda.set_device(0)
    cfg = synth.CONFIGS[args.workload]
    B, L, E = cfg.B, cfg.L, cfg.Hq * cfg.D
    p = l2a.params(B, L, L, cfg.Hq, cfg.Hkv, cfg.D, cfg.W)
    g = torch.Generator(device="cuda"); g.manual_seed(3)
    S = torch.randn((B, L, cfg.Hq, cfg.D), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    dO = torch.randn((B, L, cfg.Hq, cfg.D), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    dS = torch.empty_like(dO)
    w = torch.randn((E,), generator=g, device="cuda", dtype=torch.float32) * 0.02
    dgate = torch.randn((B, L), generator=g, device="cuda", dtype=torch.float32)
    logits = torch.empty((B, L), dtype=torch.float32, device="cuda")
    sum_sq = torch.empty((B,), dtype=torch.float32, device="cuda")
    dz = torch.empty_like(logits)
    dw = torch.empty((E,), dtype=torch.float32, device="cuda")
    dbias = torch.empty((1,), dtype=torch.float32, device="cuda")
    steps, warm = args.steps, max(3, args.warmup)
    def timed(fn):
        for _ in range(warm):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps
    ms_fwd = timed(lambda: l2a.l2a_router_logits(p, S, w, 0.0, logits, sum_sq))
    ms_bwd = timed(lambda: l2a.l2a_router_backward(p, S, w, logits, dgate, 1e-3, dO, dz, dw, dbias, dS))
    row = E * 2
    bytes_fwd, bytes_bwd = float(B * L * (row + 4)), float(B * L * (3 * row + 12))
    peak = measured_peaks()["hbm_gbs"]
    print(json.dumps({
        "metric": "L2A router kernels, achieved HBM GB/s", "value": bytes_bwd / ms_bwd / 1e6, "unit": "GB/s", "n_gpus": 1,
        "steps": steps, "warmup": warm, "ms_per_step": ms_bwd, "higher_is_better": True, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload + "_router", "B": B, "L": L, "row_elems": E,
                   "l2_policy": "S, dO and dS_loc of %.2f GB each exceed L2" % (B * L * row / 1e9)},
        "router_logits": {"ms": ms_fwd, "GB/s": bytes_fwd / ms_fwd / 1e6, "frac": bytes_fwd / ms_fwd / 1e6 / peak},
        "roofline": {"bound": "hbm", "kernel": "router_backward_kernel", "achieved": bytes_bwd / ms_bwd / 1e6, "peak": peak,
                     "unit": "GB/s", "frac": bytes_bwd / ms_bwd / 1e6 / peak, "traffic": None,
                     "algorithmic_bytes_per_launch": bytes_bwd},
        "gpu_launches": steps}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="stress_128k", choices=sorted(synth.CONFIGS))
    ap.add_argument("--density", type=float, default=None)
    ap.add_argument("--routing", default=None, choices=[None, "bernoulli", "clustered", "all", "none"])
    ap.add_argument("--forward-only", action="store_true")
    ap.add_argument("--packed-seqs", type=int, default=0,
                    help="treat the token axis as this many equal sequences packed back to back (one launch per "
                         "kernel; no end-to-end, CPU-baseline or extra legs)")
    ap.add_argument("--kv-heads", type=int, default=None,
                    help="run a slice of the workload with this many KV heads (and their query heads): small enough "
                         "for counter captures at the full sequence length")
    ap.add_argument("--shared-window", action=argparse.BooleanOptionalAction, default=False,
                    help="L2A_FLAG_SHARED_WINDOW for the headline run (default off: in the paper's layer the two modules "
                         "have their own Q/K/V; the fusion is only valid when one set feeds both, and is reported as a "
                         "labelled secondary figure)")
    ap.add_argument("--e2e-steps", type=int, default=16)
    ap.add_argument("--cpu-rows", type=int, default=96, help="rows per head of the CPU-baseline sample (0 = skip)")
    ap.add_argument("--ref-rows", type=int, default=6, help="rows per head and step of --impl reference")
    ap.add_argument("--extras", action=argparse.BooleanOptionalAction, default=True,
                    help="also time the labelled secondary figures (shared-window fusion, rho = 0.5, all routed)")
    ap.add_argument("--decode", action="store_true", help="measure the decode step instead (HBM roofline)")
    ap.add_argument("--decode-batch", type=int, default=16)
    ap.add_argument("--router", action="store_true", help="measure the router kernels instead (HBM roofline)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        return run_reference(args)
    if args.decode:
        return run_decode(args)
    if args.router:
        return run_router(args)

    from paper_2603_17484_b200 import l2a

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    cfg, rho, seed, d, logits = make_workload(args, seed_offset=rank)
    backward = not args.forward_only
    use_logits = logits is not None
    kind = l2a.ROUTER_LOGITS_F32 if use_logits else l2a.ROUTER_MASK_U8

    seq_table, seq_cu = None, None
    if args.packed_seqs > 0:
        assert cfg.B == 1, "--packed-seqs needs a single token axis"
        seq_cu = np.linspace(0, cfg.L, args.packed_seqs + 1).astype(np.int32)
        seq_table = l2a.l2a_pack_sequences(torch.from_numpy(seq_cu).cuda(), cfg.L)
        args.e2e_steps, args.cpu_rows, args.extras = 0, 0, False

    def params_for(shared):
        return l2a.params(cfg.B, cfg.L, cfg.L, cfg.Hq, cfg.Hkv, cfg.D, cfg.W, seq_bounds=seq_table,
                          flags=(l2a.FLAG_SAVE_FOR_BWD if backward else 0) | (l2a.FLAG_SHARED_WINDOW if shared else 0))

    p = params_for(args.shared_window)
    buf = l2a.Buffers.allocate(p, backward=backward, router_dtype=torch.float32 if use_logits else torch.uint8)
    if buf.lse_loc is None:      # the shared-window forward reads it back
        buf.lse_loc = torch.empty((cfg.B, cfg.Hq, cfg.L), dtype=torch.float32, device="cuda")

    # host inputs (pinned): the same seeded tensors the oracle reads
    host = {k: v.pin_memory() for k, v in synth.qkv(cfg.B, cfg.L, cfg.Hq, cfg.Hkv, cfg.D, seed, with_dO=backward).items()}
    host["router"] = torch.from_numpy(logits if use_logits else d).pin_memory()
    host["O"] = torch.empty_like(host["Q"]).pin_memory()
    if backward:
        host["dQ"] = torch.empty_like(host["Q"]).pin_memory()
        host["dK"] = torch.empty_like(host["K"]).pin_memory()
        host["dV"] = torch.empty_like(host["V"]).pin_memory()
    for name in ("Q", "K", "V") + (("dO",) if backward else ()):
        getattr(buf, name).copy_(host[name], non_blocking=True)
    buf.router.copy_(host["router"], non_blocking=True)
    torch.cuda.synchronize()

    HD = cfg.Hq * cfg.D
    per_pair = 4.0 + (10.0 if backward else 0.0)

    def pair_counts(mask):
        if seq_cu is not None:       # packed: every sequence by itself
            pl = sum(synth.pairs_local(int(e - s), cfg.W) for s, e in zip(seq_cu[:-1], seq_cu[1:]))
            pg = sum(synth.pairs_global(mask[0, s:e]) for s, e in zip(seq_cu[:-1], seq_cu[1:]))
            return pl, pg, 0
        pl = sum(synth.pairs_local(cfg.L, cfg.W) for _ in range(cfg.B))
        pg = sum(synth.pairs_global(mask[b]) for b in range(cfg.B))
        # pairs the shared-window launches do not visit: the in-window pairs of routed rows are done once, by the local items
        t = [np.nonzero(mask[b])[0].astype(np.int64) for b in range(cfg.B)]
        pw = int(sum((np.minimum(x, cfg.W) + 1).sum() for x in t))
        return pl, pg, pw

    def issued_pairs(mask, shared):
        return issued_tile_pairs(mask, cfg.L, cfg.W, shared)

    def step(profile=None):
        buf.route(kind, 0.0)
        if profile is not None:
            l2a.l2a_profile_next_call([e.cuda_event for e in profile[0]])
        buf.forward()
        if backward:
            if profile is not None:
                l2a.l2a_profile_next_call([e.cuda_event for e in profile[1]])
            buf.backward()

    def new_events(n):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        for e in ev:
            e.record()  # forces creation of the underlying handle
        return ev

    def timed_steps(n_steps, with_profile):
        prof = [(new_events(4), new_events(5)) for _ in range(n_steps)] if with_profile else [None] * n_steps
        torch.cuda.synchronize()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for i in range(n_steps):
            step(prof[i])
        stop.record()
        torch.cuda.synchronize()
        assert l2a.l2a_workspace_status(buf.fwd_ws) == 0, "device-side timeout in the forward"
        if backward:
            assert l2a.l2a_workspace_status(buf.bwd_ws) == 0, "device-side timeout in the backward"
        return start.elapsed_time(stop) / n_steps, prof

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(buf.fwd_ws) == 0, "device-side timeout in the forward"
    if backward:
        assert l2a.l2a_workspace_status(buf.bwd_ws) == 0, "device-side timeout in the backward"

    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms_local, prof = timed_steps(args.steps, True)
    clocks = sampler.stop() if rank == 0 else None
    ms_step = replicas.max_over_ranks(ms_local * args.steps, dist, "cuda") / args.steps

    # per-phase durations from the library's own stream events
    phase_ms = {}
    for names, which in ((FWD_PHASES, 0), (BWD_PHASES, 1)):
        if which == 1 and not backward:
            continue
        for k, name in enumerate(names):
            phase_ms[name] = float(np.mean([pr[which][k].elapsed_time(pr[which][k + 1]) for pr in prof]))

    pl, pg, pw = pair_counts(d)
    step_flops = per_pair * HD * (pl + pg)

    # ---- end to end through the host-buffer C-ABI call (transfers inside the timed region)
    e2e = None
    if args.e2e_steps > 0:
        # Two steps in flight on two sets of device tensors used alternately (l2a_step_host_async): the uploads of a
        # step run under the kernels of the step before it, its downloads under those of the step after it.  Every
        # step copies its inputs from pinned host memory and its results back inside the timed region, which also
        # contains the pipeline's fill (the first step's uploads are exposed) and drain.
        buf2 = l2a.Buffers.allocate(p, backward=backward, router_dtype=torch.float32 if use_logits else torch.uint8)
        if buf2.lse_loc is None:
            buf2.lse_loc = torch.empty((cfg.B, cfg.Hq, cfg.L), dtype=torch.float32, device="cuda")
        sets = (buf, buf2)
        l2a.l2a_step_host(p, host, buf, kind, 0.0)           # one blocking step, timed by itself (latency of a step)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        l2a.l2a_step_host(p, host, buf2, kind, 0.0)
        e1.record()
        torch.cuda.synchronize()
        blocking_ms = e0.elapsed_time(e1)
        if dist is not None:
            dist.barrier()
        e0.record()
        for i in range(args.e2e_steps):
            l2a.l2a_step_host_async(p, host, sets[i & 1], kind, 0.0)
        l2a.l2a_step_host_wait()
        e1.record()
        torch.cuda.synchronize()
        for b_ in sets:
            assert l2a.l2a_workspace_status(b_.fwd_ws) == 0, "device-side timeout in the host-buffer step"
        e2e_ms = replicas.max_over_ranks(e0.elapsed_time(e1) / args.e2e_steps, dist, "cuda")
        qb, kb = host["Q"].numel() * 2, host["K"].numel() * 2
        h2d = qb + 2 * kb + host["router"].numel() * host["router"].element_size() + (qb if backward else 0)
        d2h = qb + ((qb + 2 * kb) if backward else 0)
        e2e = {"value": replicas.job_throughput(world, step_flops, e2e_ms) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
               "steps": args.e2e_steps, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
               "how": "l2a_step_host_async, two steps in flight on alternating device tensors; pipeline fill and drain "
                      "inside the timed region",
               "blocking_step_ms": blocking_ms}
        del buf2, sets

    # ---- labelled secondary figures on the same tensors (rank 0 of a one-GPU run only; not the headline)
    extras = {}
    if args.extras and world == 1 and backward and args.workload == "stress_128k" and args.routing is None:
        n_x = 3

        def run_variant(mask, shared):
            buf.p = params_for(shared)
            buf.router.copy_(torch.from_numpy(mask))
            for _ in range(2):
                step()
            ms, _ = timed_steps(n_x, False)
            a, g, w = pair_counts(mask)
            return {"ms_per_step": ms, "useful_tflops": per_pair * HD * (a + g) / ms / 1e9, "density": float(mask.mean()),
                    "steps": n_x}

        if not use_logits:
            # (a) the shared-window fusion: valid only because this workload feeds ONE Q/K/V set to both modules
            extras["shared_window_fusion"] = run_variant(d, not args.shared_window)
            extras["shared_window_fusion"]["shared_window"] = not args.shared_window
            # (b) a second density, and (c) the build's own dense path (every token routed) as the internal reference
            d50 = synth.mask_clustered(cfg.B, cfg.L, 0.5, seed + 50)
            extras["density_0.5"] = run_variant(d50, args.shared_window)
            dense = run_variant(np.ones_like(d), args.shared_window)
            dense["step_time_over_dense"] = ms_step / dense["ms_per_step"]
            dense["useful_pairs_over_dense"] = (pl + pg) / (pl + sum(cfg.L * (cfg.L + 1) // 2 for _ in range(cfg.B)))
            extras["dense_reference"] = dense
            buf.p = p
            buf.router.copy_(host["router"], non_blocking=True)
            torch.cuda.synchronize()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    # Dominant kernel and its algorithmic FLOPs.  Forward kernels: 4*D per pair (local / global pairs separately); the
    # backward kernel: 10*D per pair (S, dP, dV, dK, dQ).  `achieved` credits the useful pairs of the metric; with the
    # shared-window fusion the launches do not visit the routed rows' in-window pairs of the global module (they ride on
    # the local items), so `achieved_visited` counts only the pairs the launch really processes.
    shared_now = bool(args.shared_window)
    vis_g = pg - (pw if shared_now else 0)
    kernel_pairs = {"attn_fwd_local": (4.0, pl, pl), "attn_fwd_global": (4.0, pg, vis_g), "bwd": (10.0, pl + pg, pl + vis_g)}
    tensor_phases = {k: v for k, v in phase_ms.items() if k in kernel_pairs}
    dom = max(tensor_phases, key=tensor_phases.get)
    per, credited, visited = kernel_pairs[dom]
    il, ig = issued_pairs(d, shared_now) if seq_cu is None else (credited, 0)   # (not modelled for packed batches)
    issued = {"attn_fwd_local": il, "attn_fwd_global": ig, "bwd": il + ig}[dom] if seq_cu is None else credited
    achieved = per * HD * credited / phase_ms[dom] / 1e9
    achieved_visited = per * HD * visited / phase_ms[dom] / 1e9
    # DRAM traffic of the dominant kernel: not captured on this workload (a counter capture of a 12 GB, 100 ms launch is
    # out of bounds for ncu here).  Taken from the capture of the same kernel on the 32K case (profiles/), where DRAM
    # read + write was TRAFFIC_RATIO x the launch's algorithmic bytes, and scaled by this launch's algorithmic bytes.
    qb = cfg.B * cfg.L * cfg.Hq * cfg.D * 2
    kb = cfg.B * cfg.L * cfg.Hkv * cfg.D * 2
    rho_real = float(d.mean())
    alg_bytes = {"bwd": 2 * qb * (1 + rho_real) + 4 * kb + 2 * 2 * qb * (1 + rho_real),   # Q, dO (+ compact), K, V, dK, dV, fp32 dQ acc w+r
                 "attn_fwd_local": (3 if backward else 2) * qb + 2 * kb,      # Q read, S written (twice when saving), K, V
                 "attn_fwd_global": 4 * qb * rho_real + 2 * kb}[dom]            # Q_c, A_c, routed rows of O read + written, K, V
    ratio = TRAFFIC_RATIO.get(dom)
    roofline = {"bound": "tensor", "kernel": dom, "achieved": achieved, "peak": peaks["sustained"], "unit": "TFLOP/s",
                "frac": achieved / peaks["sustained"], "traffic": ratio * alg_bytes if ratio else None,
                "traffic_source": (f"{ratio} x algorithmic bytes: ratio of the ncu capture of this kernel on the 32K case "
                                   f"(profiles/attention_kernels_qwen25_7b_32k.md), scaled to this launch") if ratio else None,
                "algorithmic_bytes_per_launch": alg_bytes,
                "peak_kind": f"sustained bf16 GEMM, {peaks['source']}", "launch_ms": phase_ms[dom],
                "algorithmic_flops_per_launch": per * HD * credited, "pairs_credited": int(credited),
                "pairs_visited": int(visited), "achieved_visited": achieved_visited,
                "frac_visited": achieved_visited / peaks["sustained"],
                # executed MMA work, tile-granular (masked elements of edge blocks and padding rows included)
                "pairs_issued": int(issued), "executed_tflops": per * HD * issued / phase_ms[dom] / 1e9}

    cpu = None
    if args.cpu_rows > 0 and world == 1:
        sm = cpu_oracle_sample(cfg, seed, d, rows_per_head=args.cpu_rows, backward=backward,
                               host={k: host[k] for k in ("Q", "K", "V") + (("dO",) if backward else ())})
        v, ext = cpu_extrapolate(cfg, d, sm, backward)
        cpu = {"value": v, "unit": "TFLOP/s", "cores": sm["cores"], "kind": "oracle", "seconds": sm["seconds"],
               "extrapolated_layer_seconds": ext,
               "pairs_per_s": {k: sm[k] for k in ("fwd_pairs_per_s", "dq_pairs_per_s", "dkv_pairs_per_s") if k in sm},
               "sample": CPU_SAMPLE_TEXT.format(rows=args.cpu_rows, heads=cfg.Hq, pr=sm["pairs_rows"], keys=8, span=2500,
                                                pk=sm.get("pairs_keys", 0), secs=sm["seconds"], ext=ext)}

    value = replicas.job_throughput(world, step_flops, ms_step) / 1e12
    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "B": cfg.B, "L": cfg.L, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
                   "W": cfg.W, "routing": args.routing or cfg.routing, "density": rho_real,
                   "pass": "fwd+bwd" if backward else "fwd", "shared_window": shared_now,
                   **({"packed_sequences": args.packed_seqs} if args.packed_seqs else {}),
                   "parallelism": f"replicas x{world}",
                   "l2_policy": "inputs larger than L2 (Q alone is %.2f GB)" % (host["Q"].numel() * 2 / 1e9),
                   "useful_tflop_per_step": step_flops / 1e12, "pairs_per_head": pl + pg,
                   "tolerance": "max |err| <= 2e-2 + 2^-8 |want|, mean |err| <= 2e-3 + 2^-9 mean |want| against the "
                                "fp64 oracle (tests/gpu_util.py)"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": KERNELS_PER_STEP * args.steps if backward else 5 * args.steps,
        "roofline": roofline, "cpu_baseline": cpu,
        "phase_ms": phase_ms,
        "frac_of_peak": {"measured_burst_%.0f" % peaks["burst"]: value / world / peaks["burst"],
                         "measured_sustained_%.0f" % peaks["sustained"]: value / world / peaks["sustained"],
                         "datasheet_2250": value / world / 2250.0},
    }
    line.update(extras)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
