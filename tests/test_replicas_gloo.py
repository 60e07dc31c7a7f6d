"""World-size-2 gloo test (CPU) of the benchmark's multi-rank logic: max-over-ranks timing and whole-job value."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_17484_b200 import replicas, synth


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    slowest = replicas.max_over_ranks(ms, dist)
    dist.barrier()
    cfg = synth.CONFIGS["tiny"]
    d0, _ = synth.routing(cfg, synth.seed_for(1) + replicas.rank_seed_offset(rank))
    out.put((rank, slowest, int(d0.sum())))
    dist.destroy_process_group()


def test_two_rank_replicas_report_slowest_time_and_sum_of_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]          # both ranks agree on the slowest time
    assert res[0][2] > 0 and res[1][2] > 0               # each replica drew its own routing mask
    assert replicas.job_throughput(2, 3.0e12, 15.0) == 2 * 3.0e12 / 15e-3
    assert replicas.max_over_ranks(7.0, None) == 7.0     # single process: identity
