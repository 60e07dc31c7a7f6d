#!/usr/bin/env python
"""Benchmark of the L2A hot path on B200: one step = route/compact + forward + backward of one layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--density RHO] [--impl reference]

Prints ONE JSON line (rank 0).  ``value`` is useful TFLOP/s with inputs resident in HBM; ``e2e`` is the
same metric through the host-buffer C-ABI call with the transfers inside the timed region;
``roofline`` describes the dominant kernel (timed with CUDA events at the phase boundaries the
library records on its own stream); ``cpu_baseline`` times the fp64 oracle on a bounded sample.
With N > 1 every rank runs an independent replica of the workload (the path has no exchange step).
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
KERNELS_PER_STEP = 11  # route: count, scan | fwd: gather, local, global | bwd: gather x2, delta, dkv, dq x2
FWD_PHASES = ("gather_q", "attn_fwd_local", "attn_fwd_global")
BWD_PHASES = ("gather_q_dO", "bwd_delta", "bwd_dq_local", "bwd_dq_global", "bwd_dkv")


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
    d, logits = synth.routing(cfg, seed, density=rho)
    return cfg, rho, seed, d, logits


def cpu_oracle_sample(cfg, seed, rho, T, backward=True):
    """fp64 oracle, forward (+ backward), on the workload truncated to its first T tokens (all heads)."""
    import oracle
    t = synth.qkv(cfg.B, T, cfg.Hq, cfg.Hkv, cfg.D, seed, with_dO=True)
    d = synth.mask_bernoulli(cfg.B, T, rho, seed) if rho < 1.0 else np.ones((cfg.B, T), np.uint8)
    sh = oracle.Shape(cfg.B, T, T, cfg.Hq, cfg.Hkv, cfg.D, cfg.W)
    Q, K, V, dO = (synth.as_u16(t[k]) for k in ("Q", "K", "V", "dO"))
    oracle.num_threads()  # builds/loads outside the timed region
    t0 = time.perf_counter()
    oracle.forward_full(sh, Q, K, V, d)
    if backward:
        oracle.backward_full(sh, Q, K, V, d, dO)
    dt = time.perf_counter() - t0
    pairs = sum(synth.pairs_local(T, cfg.W) + synth.pairs_global(d[b]) for b in range(cfg.B))
    flops = (4.0 + (10.0 if backward else 0.0)) * cfg.D * cfg.Hq * pairs
    return flops / dt / 1e12, dt, oracle.num_threads()


def run_reference(args):
    """Reference arm: the fp64 oracle as it stands on the host cores, a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, rho, seed, d, _ = make_workload(args)
    T = args.ref_tokens
    for _ in range(args.warmup):
        cpu_oracle_sample(cfg, seed, rho, min(T, 256))
    t0 = time.perf_counter()
    vals = [cpu_oracle_sample(cfg, seed + i, rho, T) for i in range(args.steps)]
    total = time.perf_counter() - t0
    value = float(np.mean([v[0] for v in vals]))
    cores = vals[0][2]
    sample = (f"fp64 oracle forward+backward on the workload truncated to its first {T} tokens (all heads, "
              f"density {rho}); the backward leg parallelises over (batch, KV head) = {cfg.B * cfg.Hkv} threads")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / max(1, args.steps) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "B": cfg.B, "L": cfg.L, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
                   "W": cfg.W, "density": rho, "sample_tokens": T},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
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


def run_paper_table(args):
    """The paper's short-context kernel table (its App. D: sparse Global Attention kernel + preprocessing at 4096 and
    8192 tokens, 28 heads, d = 128, by sparsity = 1 - routed fraction), on this build: route/compact + gather + global
    forward only (L2A_FLAG_SKIP_LOCAL), and the same with the global backward.  Context beside the paper's H200
    figures, not the headline metric; these inputs fit in L2, as they do in the paper's table."""
    from paper_2603_17484_b200 import l2a
    torch.cuda.set_device(0)
    Hq, Hkv, D = 28, 4, 128
    steps, warm = max(args.steps, 20), max(3, args.warmup)
    rows = []
    for L in (4096, 8192):
        for sparsity in (0.0, 0.2, 0.5, 0.8, 0.9, 0.95):
            d = np.ones((1, L), np.uint8) if sparsity == 0.0 else synth.mask_bernoulli(1, L, 1.0 - sparsity, seed=L + int(100 * sparsity))
            fl = l2a.FLAG_SAVE_FOR_BWD
            p_all = l2a.params(1, L, L, Hq, Hkv, D, L, flags=fl)
            buf = l2a.Buffers.allocate(p_all, backward=True)
            for t in (buf.Q, buf.K, buf.V, buf.dO):
                t.normal_()
            buf.router.copy_(torch.from_numpy(d))
            buf.route(); buf.forward()          # S_save, lse_loc for the backward call's signature
            p_glb = l2a.params(1, L, L, Hq, Hkv, D, L, flags=l2a.FLAG_SKIP_LOCAL)
            p_glb_b = l2a.params(1, L, L, Hq, Hkv, D, L, flags=fl | l2a.FLAG_SKIP_LOCAL)

            def fwd():
                buf.route()
                l2a.l2a_forward(p_glb, buf.Q, buf.K, buf.V, buf.d_mask, buf.q_idx, buf.n_routed, buf.prefix, buf.O,
                                None, None, None, None, buf.fwd_ws)

            def bwd():
                l2a.l2a_backward(p_glb_b, buf.Q, buf.K, buf.V, buf.d_mask, buf.q_idx, buf.n_routed, buf.prefix, buf.dO,
                                 None, buf.A_c, None, buf.lse_glb, buf.dQ, buf.dK, buf.dV, None, buf.bwd_ws)

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
            rows.append({"L": L, "sparsity": sparsity, "routed": int(d.sum()), "fwd_ms": timed(fwd), "bwd_ms": timed(bwd)})
            del buf
    print(json.dumps({
        "metric": "sparse Global Attention kernel + preprocessing, short contexts (paper's kernel table)", "unit": "ms",
        "value": rows[-1]["fwd_ms"], "n_gpus": 1, "steps": steps, "warmup": warm, "higher_is_better": False,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "paper_kernel_table", "B": 1, "Hq": Hq, "Hkv": Hkv, "D": D,
                   "l2_policy": "inputs fit in L2, as in the paper's table; no flush",
                   "note": "forward = route/compact + gather + global forward; backward = global backward of the same rows"},
        "rows": rows, "gpu_launches": 4 * steps}), flush=True)


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
    ap.add_argument("--shared-window", action=argparse.BooleanOptionalAction, default=True,
                    help="L2A_FLAG_SHARED_WINDOW (default on: every workload here feeds one Q/K/V set to both "
                         "modules): global attention reuses the local pass for the keys inside the window; "
                         "--no-shared-window runs the two modules independently")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--cpu-tokens", type=int, default=2048, help="tokens of the CPU-baseline sample (0 = skip)")
    ap.add_argument("--ref-tokens", type=int, default=1024, help="tokens per step of --impl reference")
    ap.add_argument("--decode", action="store_true", help="measure the decode step instead (HBM roofline)")
    ap.add_argument("--decode-batch", type=int, default=16)
    ap.add_argument("--router", action="store_true", help="measure the router kernels instead (HBM roofline)")
    ap.add_argument("--paper-table", action="store_true",
                    help="the paper's short-context kernel table on this build (context, not the headline)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        return run_reference(args)
    if args.decode:
        return run_decode(args)
    if args.router:
        return run_router(args)
    if args.paper_table:
        return run_paper_table(args)

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
    flags = (l2a.FLAG_SAVE_FOR_BWD if backward else 0) | (l2a.FLAG_SHARED_WINDOW if args.shared_window else 0)
    p = l2a.params(cfg.B, cfg.L, cfg.L, cfg.Hq, cfg.Hkv, cfg.D, cfg.W, flags=flags)
    use_logits = logits is not None
    buf = l2a.Buffers.allocate(p, backward=backward, router_dtype=torch.float32 if use_logits else torch.uint8)
    if args.shared_window and not backward:
        buf.lse_loc = torch.empty((cfg.B, cfg.Hq, cfg.L), dtype=torch.float32, device="cuda")
    kind = l2a.ROUTER_LOGITS_F32 if use_logits else l2a.ROUTER_MASK_U8

    # host inputs (pinned): the same seeded tensors the oracle would read
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

    fwd_flops, bwd_flops = synth.useful_flops(cfg, d, backward)
    pairs = sum(synth.pairs_local(cfg.L, cfg.W) + synth.pairs_global(d[b]) for b in range(cfg.B))
    step_flops = fwd_flops + bwd_flops

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

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert l2a.l2a_workspace_status(buf.fwd_ws) == 0, "device-side timeout in the forward"
    if backward:
        assert l2a.l2a_workspace_status(buf.bwd_ws) == 0, "device-side timeout in the backward"

    prof = [(new_events(4), new_events(6)) for _ in range(args.steps)]
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record()
    for i in range(args.steps):
        step(prof[i])
    stop.record()
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = replicas.max_over_ranks(start.elapsed_time(stop), dist, "cuda")
    ms_step = ms_total / args.steps

    # per-phase durations from the library's own stream events
    phase_ms = {}
    for names, which in ((FWD_PHASES, 0), (BWD_PHASES, 1)):
        if which == 1 and not backward:
            continue
        for k, name in enumerate(names):
            phase_ms[name] = float(np.mean([pr[which][k].elapsed_time(pr[which][k + 1]) for pr in prof]))

    # ---- end to end through the host-buffer C-ABI call (transfers inside the timed region)
    e2e = None
    if args.e2e_steps > 0:
        l2a.l2a_step_host(p, host, buf, kind, 0.0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        e0.record()
        for _ in range(args.e2e_steps):
            l2a.l2a_step_host(p, host, buf, kind, 0.0)
        e1.record()
        torch.cuda.synchronize()
        e2e_ms = replicas.max_over_ranks(e0.elapsed_time(e1) / args.e2e_steps, dist, "cuda")
        qb, kb = host["Q"].numel() * 2, host["K"].numel() * 2
        h2d = qb + 2 * kb + host["router"].numel() * host["router"].element_size() + (qb if backward else 0)
        d2h = qb + ((qb + 2 * kb) if backward else 0)
        e2e = {"value": replicas.job_throughput(world, step_flops, e2e_ms) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    # dominant kernel and its algorithmic FLOPs: forward kernels 4*D per pair (local / global pairs
    # separately); dK/dV kernel 8*D per pair (S, dP, dV, dK); dQ kernels 2*D per pair (dQ only; their
    # recomputation of S and dP is not algorithmic work)
    HD = cfg.Hq * cfg.D
    pl = sum(synth.pairs_local(cfg.L, cfg.W) for _ in range(cfg.B))
    pg = sum(synth.pairs_global(d[b]) for b in range(cfg.B))
    kernel_flops = {"attn_fwd_local": 4.0 * HD * pl, "attn_fwd_global": 4.0 * HD * pg,
                    "bwd_dkv": 8.0 * HD * (pl + pg), "bwd_dq_local": 2.0 * HD * pl, "bwd_dq_global": 2.0 * HD * pg}
    tensor_phases = {k: v for k, v in phase_ms.items() if k in kernel_flops}
    dom = max(tensor_phases, key=tensor_phases.get)
    achieved = kernel_flops[dom] / phase_ms[dom] / 1e9
    # DRAM traffic of the dominant kernel.  Measured with ncu (one pass, dram__bytes_read.sum + dram__bytes_write.sum)
    # on this very workload, stress_128k: 4.57 GB read + 0.56 GB written per dK/dV launch = 1.42 x the algorithmic
    # bytes of the launch (Q, dO and their compact copies read once, K and V read, dK and dV written); on the 32K
    # case the ratio is 1.13 (profiles/).  Other workloads report the figure scaled by their tensor bytes.
    qb = cfg.B * cfg.L * cfg.Hq * cfg.D * 2
    kb = cfg.B * cfg.L * cfg.Hkv * cfg.D * 2
    dkv_alg_bytes = 2 * qb * (1 + float(d.mean())) + 4 * kb
    traffic = (1.42 if cfg.L > 65536 else 1.13) * dkv_alg_bytes if dom == "bwd_dkv" else None
    roofline = {"bound": "tensor", "kernel": dom, "achieved": achieved, "peak": peaks["sustained"], "unit": "TFLOP/s",
                "frac": achieved / peaks["sustained"], "traffic": traffic,
                "traffic_note": "bytes per launch: ncu capture of the 128K workload (1.42 x algorithmic bytes) or of the "
                                "32K case (1.13 x), scaled by the launch's tensor bytes",
                "peak_kind": f"sustained bf16 GEMM, {peaks['source']}", "launch_ms": phase_ms[dom],
                "algorithmic_flops_per_launch": kernel_flops[dom]}

    cpu = None
    if args.cpu_tokens > 0 and world == 1:
        v, dt, cores = cpu_oracle_sample(cfg, seed, min(rho, 1.0), args.cpu_tokens, backward)
        cpu = {"value": v, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "seconds": dt,
               "sample": f"fp64 oracle {'forward+backward' if backward else 'forward'} on the workload truncated to "
                         f"its first {args.cpu_tokens} tokens (all heads, Bernoulli density {rho}); the backward leg "
                         f"parallelises over (batch, KV head) = {cfg.B * cfg.Hkv} threads"}

    value = replicas.job_throughput(world, step_flops, ms_step) / 1e12
    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "B": cfg.B, "L": cfg.L, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
                   "W": cfg.W, "routing": args.routing or cfg.routing, "density": float(d.mean()),
                   "pass": "fwd+bwd" if backward else "fwd", "shared_window": bool(args.shared_window),
                   "parallelism": f"replicas x{world}",
                   "l2_policy": "inputs larger than L2 (Q alone is %.2f GB)" % (host["Q"].numel() * 2 / 1e9),
                   "useful_tflop_per_step": step_flops / 1e12, "pairs_per_head": pairs},
        "clocks": clocks, "e2e": e2e, "gpu_launches": KERNELS_PER_STEP * args.steps if backward else 5 * args.steps,
        "roofline": roofline, "cpu_baseline": cpu,
        "phase_ms": phase_ms,
        "frac_of_peak": {"measured_burst_%.0f" % peaks["burst"]: value / world / peaks["burst"],
                         "measured_sustained_%.0f" % peaks["sustained"]: value / world / peaks["sustained"],
                         "datasheet_2250": value / world / 2250.0},
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
