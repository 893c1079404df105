"""Host-side logic of the multi-GPU run (independent replicas, no collective in the step), exercised with two
gloo ranks on the CPU: disjoint sample-index ranges per rank, MAX-over-ranks timing, whole-job throughput."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    B, steps = 4096, 10
    plan = bench.rank_plan(rank, world, B)
    local_ms = 100.0 + 50.0 * rank                       # rank 1 is the slow one
    dist.barrier()
    ms_max = bench.max_over_ranks(local_ms, world)        # CPU tensor, gloo
    gathered = [None] * world
    dist.all_gather_object(gathered, plan)
    if rank == 0:
        out.put((ms_max, gathered, bench.whole_job_value(world, B, steps, ms_max)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_replica_plan_and_timing():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    ms_max, plans, value = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ms_max == 150.0                               # the slowest rank's time, seen by rank 0
    assert plans[0]["sample_idx_base"] == 0 and plans[1]["sample_idx_base"] == 4096
    assert plans[0]["last_sample"] + 1 == plans[1]["first_sample"]          # contiguous, disjoint
    assert plans[1]["last_sample"] + 1 == plans[0]["total_samples"] == 8192
    assert value == 2 * 4096 * 10 / 0.150


def test_single_rank_is_the_identity():
    import bench
    assert bench.max_over_ranks(12.5, 1) == 12.5
    assert bench.rank_plan(0, 1, 7) == {"sample_idx_base": 0, "first_sample": 0, "last_sample": 6, "total_samples": 7}
    assert bench.whole_job_value(1, 100, 3, 1.0) == 300000.0
