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
    import socket
    with socket.socket() as sk:                          # a port that is free right now
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
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


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` with WORLD_SIZE unset starts two local ranks itself. On a box without a GPU
    the ranks must stop with the no-CUDA message (there is no CPU fallback) and the command must fail, rather
    than one rank running silently as a 1-GPU job. (The launcher ends the other rank as soon as the first one has
    failed, so the second message may or may not appear; a message of a rank that cannot exist must not.)"""
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode != 0
    text = res.stdout + res.stderr
    assert "rank 0: bench.py needs a CUDA device" in text or "rank 1: bench.py needs a CUDA device" in text
    assert "rank 2:" not in text
    assert '"n_gpus"' not in res.stdout                    # no result line was printed


def test_a_rank_count_that_contradicts_the_flag_is_refused():
    import subprocess
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0", CUDA_VISIBLE_DEVICES="")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode != 0 and "--gpus 2 but the launcher started 1 rank" in res.stderr


def test_traffic_figure_is_read_from_the_profile_summaries_and_dropped_when_the_kernel_changed(tmp_path, monkeypatch):
    """bench.py takes the DRAM traffic of the dominant kernel from a line in profiles/*.md that names workload, batch
    and the hash of the GEMM sources it was captured on; no line, another batch or another hash give None."""
    import bench
    (tmp_path / "profiles").mkdir()
    (tmp_path / "profiles" / "x.md").write_text(
        "text\n    dram_traffic_per_step: workload=mid batch=4096 bytes=1.25e9 gemm_sources=abc123\nmore\n")
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    monkeypatch.setattr(bench, "gemm_sources_sha", lambda: "abc123")
    assert bench.dram_traffic_per_step("mid", 4096) == 1.25e9
    assert bench.dram_traffic_per_step("mid", 8192) is None and bench.dram_traffic_per_step("rl", 4096) is None
    monkeypatch.setattr(bench, "gemm_sources_sha", lambda: "fff000")
    assert bench.dram_traffic_per_step("mid", 4096) is None
