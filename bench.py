#!/usr/bin/env python
"""Benchmark of the SRM decode hot path on B200: generated tokens/s at a given batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload mid] [--batch B]
    python bench.py --impl reference ...      # the CPU oracle on the host cores, same metric
    python bench.py --sweep                   # tokens/s-vs-batch curve + maximum concurrency

A "step" is one recurrent decode step of the whole batch: embedding, L x (fused token-mixer
state update + feed-forward up/down GEMMs), final norm, LM head, token selection. The
sequence-parallel prefill that builds the cache runs once before the timed region and is timed
and reported separately ("prefill"). One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC, UNIT = "generated_tokens_per_s", "tokens/s"
L2_BYTES = 126e6
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
MIN_TIMED_S = 1.0          # a K-step block is repeated until this much device time has been timed


def gemm_sources_sha():
    """Short hash of the tensor-core GEMM sources: a DRAM-traffic figure taken under ncu holds only for the
    kernel it was taken on."""
    import hashlib
    h = hashlib.sha256()
    for f in ("gemm_tc.cuh", "gemm_tc_splitk.cuh", "ffn_fused.cuh", "ffn_plan.h"):
        with open(os.path.join(ROOT, "paper_2605_08696_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:12]


def dram_traffic_per_step(workload: str, batch: int):
    """DRAM bytes (read + write) of the GEMM launches of one decode step, from the ncu summaries under profiles/:
    a line `dram_traffic_per_step: workload=<w> batch=<B> bytes=<x> gemm_sources=<sha>`. None when no capture
    exists for this workload and batch, or when the GEMM sources have changed since it was taken."""
    import glob
    import re
    pat = re.compile(r"dram_traffic_per_step:\s*workload=(\w+)\s+batch=(\d+)\s+bytes=([0-9.eE+]+)\s+gemm_sources=(\w+)")
    sha = gemm_sources_sha()
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.md"))):
        with open(path) as f:
            for m in pat.finditer(f.read()):
                if m.group(1) == workload and int(m.group(2)) == batch and m.group(4) == sha:
                    return float(m.group(3))
    return None


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock, power and clock-event (throttle) reasons of one GPU every ~10 ms while the timed
    regions run: NVML queries from a thread of this process (read-only), or an `nvidia-smi` loop when NVML
    cannot be loaded. Only samples that fall inside a marked region are summarised."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    PERIOD_S = 0.010

    def __init__(self, index: int, uuid: str | None = None):
        self.index, self.uuid = index, uuid
        self.rows = []            # (monotonic time, sm MHz, max MHz, watts, set of reasons)
        self.regions = []         # [t0, t1] of the marked regions
        self.proc = self.thread = self.nvml = None
        self.stop = threading.Event()
        self.source = None

    # -- regions --
    def mark_start(self):
        self.regions.append([time.monotonic(), None])

    def mark_stop(self):
        self.regions[-1][1] = time.monotonic()

    # -- NVML --
    def _nvml_open(self):
        import pynvml
        pynvml.nvmlInit()
        h = None
        if self.uuid:
            for u in (self.uuid, "GPU-" + self.uuid):
                try:
                    h = pynvml.nvmlDeviceGetHandleByUUID(u if isinstance(u, bytes) else u.encode())
                    break
                except Exception:
                    h = None
        if h is None:
            h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
        self.nvml, self.h = pynvml, h
        self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        n = pynvml
        self.bits = [(getattr(n, "nvmlClocksEventReasonSwPowerCap", 0x4), "sw_power_cap"),
                     (getattr(n, "nvmlClocksThrottleReasonHwSlowdown", 0x8), "hw_slowdown"),
                     (getattr(n, "nvmlClocksEventReasonSwThermalSlowdown", 0x20), "sw_thermal_slowdown"),
                     (getattr(n, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40), "hw_thermal_slowdown")]

    def _nvml_loop(self):
        n, h = self.nvml, self.h
        get_reasons = getattr(n, "nvmlDeviceGetCurrentClocksEventReasons", None) or n.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self.stop.is_set():
            try:
                mhz = float(n.nvmlDeviceGetClockInfo(h, n.NVML_CLOCK_SM))
                mask = int(get_reasons(h))
                watts = n.nvmlDeviceGetPowerUsage(h) / 1000.0
                self.rows.append((time.monotonic(), mhz, self.max_mhz, watts,
                                  {name for bit, name in self.bits if mask & bit}))
            except Exception:
                pass
            time.sleep(self.PERIOD_S)

    # -- nvidia-smi fallback --
    def _smi_loop(self):
        for line in self.proc.stdout:
            r = [c.strip() for c in line.split(",")]
            if len(r) < 8:
                continue
            try:
                mhz, mx, watts = float(r[0]), float(r[1]), float(r[2])
            except ValueError:
                continue
            reasons = {name for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4:8])
                       if v.lower().startswith("active")}
            self.rows.append((time.monotonic(), mhz, mx, watts, reasons))

    def __enter__(self):
        try:
            self._nvml_open()
            self.thread = threading.Thread(target=self._nvml_loop, daemon=True)
            self.source = "nvml, 10 ms"
        except Exception:
            self.nvml = None
            try:
                self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                              "--format=csv,noheader,nounits", "-lms", "20"],
                                             stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
                self.thread = threading.Thread(target=self._smi_loop, daemon=True)
                self.source = "nvidia-smi, 20 ms"
            except OSError:
                self.proc = self.thread = None
        if self.thread is not None:
            self.thread.start()
        return self

    def __exit__(self, *a):
        self.stop.set()
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)
        if self.nvml is not None:
            try:
                self.nvml.nvmlShutdown()
            except Exception:
                pass

    def summary(self, regions=None):
        """Median SM clock, maximum clock, reasons seen and sample count over the marked regions (or the given
        [t0, t1] pairs)."""
        regions = self.regions if regions is None else regions
        inside = [r for r in self.rows if any(t0 <= r[0] <= (t1 if t1 is not None else r[0]) for t0, t1 in regions)]
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "source": self.source}
        reasons = set().union(*[r[4] for r in inside])
        return {"sm_mhz": statistics.median(r[1] for r in inside), "sm_max_mhz": max(r[2] for r in inside),
                "sm_mhz_min": min(r[1] for r in inside), "power_w": round(statistics.median(r[3] for r in inside), 1),
                "reasons": sorted(reasons), "samples": len(inside), "source": self.source}


def step_flops(shape):
    d, L, V = shape.d_model, shape.n_layers, shape.vocab
    per_layer = 20 if shape.head_proj else 16    # FFN up + down (16 d^2), head projections W_in + W_out (4 d^2)
    return per_layer * L * d * d + 2 * d * V     # per generated token


def step_roofline_s(shape, B, state_bytes, peaks):
    """Slower of the step's FLOPs at the tensor peak and its weight + state bytes at HBM bandwidth."""
    d, L, V = shape.d_model, shape.n_layers, shape.vocab
    t_tc = B * step_flops(shape) / (peaks["bf16_tflops_sustained"] * 1e12)
    bytes_ = step_flops(shape) + B * 2 * L * d * state_bytes      # bf16 weights: as many bytes as flop per token
    t_hbm = bytes_ / (peaks["hbm_gbs"] * 1e9)
    return max(t_tc, t_hbm), ("tensor" if t_tc >= t_hbm else "hbm"), t_tc, t_hbm


# ----------------------------------------------------------------------------------------------
def run_reference(args):
    """The CPU oracle (numpy fp64, as it stands) on the host cores: same metric and config, each
    step a bounded sample of the batch."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import srm_inputs as I
    from oracle import srm_oracle as O
    w = I.WORKLOADS[args.workload]
    shape = I.CONFIGS[w["model"]]
    if args.head_proj:
        import dataclasses
        shape = dataclasses.replace(shape, head_proj=True)
    B_full = args.batch or w["batch"] or 4096
    sample = min(B_full, args.ref_samples)
    W = I.make_weights(shape)
    orc = O.SRMOracle(shape.n_layers, shape.d_model, shape.vocab, shape.n_ctx, W, n_heads=shape.n_heads,
                      ln_eps=shape.ln_eps)
    rng = np.random.default_rng(0)
    state = rng.normal(size=(shape.n_layers, sample, shape.d_model))
    tok = I.make_prompts(args.workload, batch=sample)[:, 0]
    pos = w["prompt_len"]
    for _ in range(args.warmup):
        lg, state = orc.decode_step(state, tok, pos); tok = O.select_greedy(lg); pos += 1
    t0 = time.perf_counter()
    for _ in range(args.steps):
        lg, state = orc.decode_step(state, tok, pos); tok = O.select_greedy(lg)
        pos = pos + 1 if pos + 1 < shape.n_ctx else w["prompt_len"]
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    cores = _blas_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": _config_dict(args, shape, w, B_full, extra={"sample": f"{sample} of {B_full} samples per step"}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{sample} samples x {args.steps} decode steps (numpy fp64 oracle)"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def _blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count()


def _config_dict(args, shape, w, B, extra=None):
    mix = {"mixed": "", "combined": " + combined heads", "kernel": f" + kernels of size {shape.kernel_size}"}[shape.mixer]
    c = {"workload": f"{args.workload}{' + head projections' if shape.head_proj else ''}{mix}: SRM L{shape.n_layers} d{shape.d_model} F{shape.d_ffn} V{shape.vocab} "
                     f"n_ctx{shape.n_ctx} {shape.dtype}, batch {B}, prompts {w['prompt_len']} tokens ({w['prompts']}), "
                     f"{w['sampling']} selection",
         "batch_per_gpu": B, "prompt_len": w["prompt_len"], "selection": w["sampling"],
         "parallelism": "independent replicas, no collective"}
    if extra:
        c.update(extra)
    return c


def cpu_baseline(shape, W, workload, w, seconds_target=12.0):
    """Times the oracle's decode step on a bounded sample on the host cores."""
    import numpy as np
    import srm_inputs as I
    from oracle import srm_oracle as O
    orc = O.SRMOracle(shape.n_layers, shape.d_model, shape.vocab, shape.n_ctx, W, n_heads=shape.n_heads,
                      ln_eps=shape.ln_eps)
    sample = 32
    state = np.random.default_rng(0).normal(size=(shape.n_layers, sample, shape.d_model))
    tok = I.make_prompts(workload, batch=sample)[:, 0]
    pos = w["prompt_len"]
    lg, state = orc.decode_step(state, tok, pos)            # warm-up (BLAS threads, page faults)
    steps, t0 = 0, time.perf_counter()
    while True:
        lg, state = orc.decode_step(state, tok, pos + 1 + steps % 8)
        tok = O.select_greedy(lg)
        steps += 1
        dt = time.perf_counter() - t0
        if dt > seconds_target or steps >= 512:
            break
    return {"value": sample * steps / dt, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle",
            "sample": f"{sample} samples x {steps} decode steps of the same model (numpy fp64 oracle, {dt:.1f} s)"}


# ---- multi-GPU: independent replicas, no collective in the step -------------------------------
def rank_plan(rank: int, world: int, B: int) -> dict:
    """What differs between the replicas: each rank owns B samples of the whole job, global sample
    indices [rank*B, (rank+1)*B) (they key the Philox draws), and runs the same step on its own GPU."""
    return {"sample_idx_base": rank * B, "first_sample": rank * B, "last_sample": (rank + 1) * B - 1,
            "total_samples": world * B}


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Device-timed duration of the slowest rank (MAX all-reduce; identity for one rank)."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.item()


def whole_job_value(world: int, B: int, steps: int, ms_max: float) -> float:
    """tokens/s of the whole job: every rank generated B tokens per step, the job took the slowest rank's time."""
    return world * B * steps / (ms_max / 1e3)


# ----------------------------------------------------------------------------------------------
def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2605_08696_b200 as P
    import srm_inputs as I

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {world} rank(s)")
    if not torch.cuda.is_available():
        raise SystemExit(f"rank {rank}: bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    w = I.WORKLOADS[args.workload]
    if args.top_p is not None:         # nucleus sampling instead of the workload's selection rule
        w = dict(w, sampling="topp", top_p=args.top_p, temperature=args.temperature or 0.7)
    shape = I.CONFIGS[w["model"]]
    import dataclasses
    if args.head_proj:
        shape = dataclasses.replace(shape, head_proj=True)
    if args.mixer != "mixed":
        shape = dataclasses.replace(shape, mixer=args.mixer, kernel_size=args.kernel_size if args.mixer == "kernel" else 1)
    planes = {"mixed": 1, "combined": 2, "kernel": args.kernel_size}[args.mixer]     # d-vectors of cache per sample and layer
    B = args.batch or w["batch"] or 4096
    n = w["prompt_len"]
    peaks, peak_src = measured_peaks()

    W = I.make_weights(shape)
    model = P.SRM(shape, W, device=dev, state_dtype=args.state_dtype,
                  flags={"auto": 0, "on": P.FLAG_GRAPH, "off": P.FLAG_NO_GRAPH}[args.graph] |
                  (P.FLAG_NO_SPLITK if args.no_splitk else 0) | (P.FLAG_NO_TAIL_SPLIT if args.no_tail_split else 0) |
                  (P.FLAG_NO_FUSED_FFN if args.no_fused_ffn else 0) | (P.FLAG_NO_KSLICE if args.no_kslice else 0) |
                  (P.FLAG_NO_SMALL_BATCH if args.no_small_batch else 0))
    sidx0 = rank_plan(rank, world, B)["sample_idx_base"]
    samp = {"greedy": lambda: P.Sampling("greedy"),
            "topk": lambda: P.Sampling("topk", w["top_k"], w["temperature"], seed=shape.seed, sample_idx_base=sidx0),
            "topp": lambda: P.Sampling("topp", temperature=w["temperature"], seed=shape.seed, sample_idx_base=sidx0,
                                       top_p=w["top_p"])}[w["sampling"]]()
    prompts = torch.from_numpy(I.make_prompts(args.workload, batch=B)).to(dev)
    chunk = min(B, args.chunk)
    st = model.new_state(B)
    ws = model.new_workspace(chunk, n, prefill_samples=max(1, min(B, args.prefill_rows // n)))
    sbytes = 4 if args.state_dtype == "fp32" else 2

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- prefill (once; timed separately) ----
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    prefill_ms = None
    lengths = None
    if args.ragged:                          # a serving mix: prompt lengths uniform on [n/2, n], one position per sample
        import numpy as np
        rng = np.random.Generator(np.random.Philox(key=shape.seed + 77))
        lengths = torch.from_numpy(rng.integers(n // 2, n + 1, size=B).astype(np.int32)).to(dev)
        if args.no_prefill:
            raise SystemExit("--ragged needs the prefill (it sets the per-sample positions)")
    if args.no_prefill:                      # profiling aid: decode cost does not depend on the cache contents
        st.pos = n
    else:
        replicated = w["prompts"] == "replicated" and B % w["n_prompts"] == 0 and not args.no_prompt_dedup

        def do_prefill():
            if lengths is not None:
                model.prefill_ragged(st, prompts, lengths, samp, ws)
            elif replicated:                   # each distinct prompt runs once, its cache is copied to its replicas
                reps = B // w["n_prompts"]
                model.prefill_replicated(st, prompts[::reps].contiguous(), reps, samp, ws)
            else:
                model.prefill(st, prompts, samp, ws)

        do_prefill()                         # untimed: first-use costs (module load, descriptor encoding)
        st.reset()
        torch.cuda.synchronize()
        e0.record()
        do_prefill()
        e1.record()
        torch.cuda.synchronize()
        prefill_ms = e0.elapsed_time(e1)

    def rewind():
        """Back to the end of the prompt when the context is exhausted (timing only: alpha/beta indices stay in
        range). Per-sample positions live on the device, so a ragged state is prefilled again instead."""
        if lengths is not None:
            st.reset()
            do_prefill()
        else:
            st.pos = n

    step_no = [1]
    store = torch.empty(B, shape.n_ctx - n, dtype=torch.int32, device=dev)       # generated-token store

    def run_steps(k):
        """k decode steps through the generation loop of the library (srm_generate: launch by launch, or a
        replayed CUDA graph for launch-bound batches); the position wraps to the end of the prompt when the
        context is exhausted (timing only: alpha/beta indices stay in range)."""
        while k > 0:
            room = shape.n_ctx - st.pos
            if room == 0:
                rewind()
                continue
            c = min(k, room)
            model.generate(st, c, step_no[0], samp, ws, out=store)
            step_no[0] += c
            k -= c

    def timed_blocks(run_block, clk):
        """Times run_block (EXACTLY K steps) between a barrier + synchronize on both sides, MAX over ranks, and
        repeats the block until MIN_TIMED_S of device time has been timed: a single 20-step block lasts tens of
        milliseconds, which measures the clock transient after the prefill, not the kernels. Every rank
        computes the same number of blocks from the first block's MAX-over-ranks time."""
        times, n_target = [], None
        while n_target is None or len(times) < n_target:
            sync_all()
            clk.mark_start()
            e0.record()
            run_block()
            e1.record()
            torch.cuda.synchronize()
            clk.mark_stop()
            times.append(max_over_ranks(e0.elapsed_time(e1), world, dev))
            if n_target is None:
                n_target = max(1, min(args.max_blocks, math.ceil(args.min_time * 1e3 / max(times[0], 1e-3))))
        return times

    try:
        uuid = str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        uuid = None
    with ClockSampler(local, uuid) as clk:
        run_steps(max(args.warmup, 3))
        # ---- timed region: blocks of exactly K steps ----
        sync_all()
        launches0 = model.kernel_launches()
        run_steps(args.steps)                # one more untimed block, to count the launches of K steps
        torch.cuda.synchronize()
        launches = model.kernel_launches() - launches0
        block_ms = timed_blocks(lambda: run_steps(args.steps), clk)
        timed_regions = list(clk.regions)
    t_ms_max = statistics.median(block_ms)
    value = whole_job_value(world, B, args.steps, t_ms_max)

    # ---- per-kernel durations, CUDA events on the launching stream, same workload ----
    if lengths is not None and shape.n_ctx - st.pos < args.steps:
        rewind()
    prof_steps = args.steps * max(1, min(len(block_ms), 256 // max(args.steps, 1)))   # long enough to sit at the
    model.profile_reset()                                                              # same clocks, bounded events
    model.profile(True)
    run_steps(prof_steps)
    torch.cuda.synchronize()
    model.profile(False)
    prof = model.profile_read()
    d, L, V, F = shape.d_model, shape.n_layers, shape.vocab, shape.d_ffn
    single_kernel = prof["step_small"][0] > 0          # small batch: the whole step is one kernel (dense work included)
    gemm_classes = ("step_small",) if single_kernel else ("ffn", "gemm_up", "gemm_down", "gemm_lm", "gemm_proj")
    gemm_ms = sum(prof[k][1] for k in gemm_classes)
    gemm_launches = sum(prof[k][0] for k in gemm_classes)
    gemm_flops = prof_steps * B * step_flops(shape)
    achieved_tf = gemm_flops / (gemm_ms / 1e3) / 1e12 if gemm_ms > 0 else 0.0
    prof_total = sum(v[1] for v in prof.values())
    peak_tf = peaks["bf16_tflops_sustained"]
    t_roof, bound, t_tc, t_hbm = step_roofline_s(shape, B, sbytes * planes, peaks)
    mixer_bytes = prof_steps * L * B * d * (4 + 4 + 2 * sbytes * planes + 2)       # x r/w, cache r/w, bf16 activation
    mixer_cache_bytes = prof_steps * L * B * d * 2 * sbytes * planes                # the part that must cross HBM: cache read + write
    kernels = {k: {"launches": v[0], "ms_total": round(v[1], 3), "share": round(v[1] / prof_total, 4) if prof_total else 0}
               for k, v in prof.items() if v[0]}
    if not single_kernel:
        if "ffn" in kernels:             # up and down projection of a layer in one kernel
            kernels["ffn"]["tflops"] = round(prof_steps * L * B * 4 * d * F / (prof["ffn"][1] / 1e3) / 1e12, 1)
        if "gemm_up" in kernels:
            kernels["gemm_up"]["tflops"] = round(prof_steps * L * B * 2 * d * F / (prof["gemm_up"][1] / 1e3) / 1e12, 1)
            kernels["gemm_down"]["tflops"] = round(prof_steps * L * B * 2 * d * F / (prof["gemm_down"][1] / 1e3) / 1e12, 1)
        kernels["gemm_lm"]["tflops"] = round(prof_steps * B * 2 * d * V / (prof["gemm_lm"][1] / 1e3) / 1e12, 1)
        if shape.head_proj:
            kernels["gemm_proj"]["tflops"] = round(prof_steps * L * B * 4 * d * d / (prof["gemm_proj"][1] / 1e3) / 1e12, 1)
        kernels["mixer"]["gbs"] = round(mixer_bytes / (prof["mixer"][1] / 1e3) / 1e9, 1)          # all bytes it moves (x and a: L2)
        kernels["mixer"]["cache_gbs"] = round(mixer_cache_bytes / (prof["mixer"][1] / 1e3) / 1e9, 1)   # algorithmic: the cache
        kernels["mixer"]["cache_frac_of_hbm_peak"] = round(kernels["mixer"]["cache_gbs"] / peaks["hbm_gbs"], 3)
    else:                                # bound by reading the weights once per step
        kernels["step_small"]["weight_gbs"] = round(prof_steps * step_flops(shape) / (prof["step_small"][1] / 1e3) / 1e9, 1)
        kernels["step_small"]["frac_of_hbm_peak"] = round(kernels["step_small"]["weight_gbs"] / peaks["hbm_gbs"], 3)
    for k_ in kernels.values():
        k_["us_per_launch"] = round(k_["ms_total"] * 1e3 / k_["launches"], 2)
    if samp.mode != "greedy" and "select" in kernels:   # greedy selection is fused into the LM head: nothing to rate
        kernels["select"]["gbs"] = round(prof_steps * B * V * 4 / (prof["select"][1] / 1e3) / 1e9, 1)

    # ---- end to end through the host-buffer call: H2D tokens in, D2H tokens out, every step ----
    if lengths is not None and shape.n_ctx - st.pos < args.steps + 2:
        rewind()
    h_in = st.last_token().cpu().pin_memory()
    h_out = torch.empty_like(h_in).pin_memory()
    for _ in range(2):
        if st.pos >= shape.n_ctx:
            rewind()
        model.decode_step_host(st, h_in, samp, step_no[0], h_out, ws); step_no[0] += 1
        torch.cuda.synchronize(); h_in.copy_(h_out)

    def e2e_block():
        for _ in range(args.steps):
            if st.pos >= shape.n_ctx:
                rewind()
            model.decode_step_host(st, h_in, samp, step_no[0], h_out, ws); step_no[0] += 1
            torch.cuda.current_stream().synchronize()      # the next step's input is this step's output
            h_in.copy_(h_out)

    with ClockSampler(local, uuid) as clk2:
        e2e_ms = timed_blocks(e2e_block, clk2)
        e2e_clocks = clk2.summary()
    e2e_value = whole_job_value(world, B, args.steps, statistics.median(e2e_ms))
    status = st.status()

    if single_kernel:
        # the step is one weight-streaming kernel: algorithmic bytes = the bf16 weights once + the cache read and written
        step_bytes = step_flops(shape) + B * 2 * L * d * sbytes
        gbs = prof_steps * step_bytes / (gemm_ms / 1e3) / 1e9 if gemm_ms > 0 else 0.0
        roofline = {"bound": "hbm", "kernel": "step_small_kernel (the whole decode step of a batch of at most 64 samples)",
                    "achieved": round(gbs, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(gbs / peaks["hbm_gbs"], 4),
                    "peak_source": f"hbm_gbs, {peak_src}", "launches": int(gemm_launches), "steps_profiled": prof_steps,
                    "traffic": None, "bytes_per_step": step_bytes}
    else:
        roofline = {"bound": "tensor", "kernel": "ffn_fused_kernel + gemm_tc_kernel (feed-forward up/down + LM head)" if prof["ffn"][0] else "gemm_tc_kernel (feed-forward up/down + LM head)",
                    "achieved": round(achieved_tf, 1), "peak": peak_tf, "unit": "TFLOP/s",
                    "frac": round(achieved_tf / peak_tf, 4), "peak_source": f"bf16_tflops_sustained, {peak_src}",
                    "frac_of_burst_peak": round(achieved_tf / peaks["bf16_tflops"], 4),
                    "launches": int(gemm_launches), "steps_profiled": prof_steps,
                    "traffic": dram_traffic_per_step(args.workload, B) if not (shape.head_proj or planes > 1) else None,
                    "traffic_note": "DRAM bytes of the GEMM launches of one step (ncu, cold cache; see profiles/); "
                                    "null when no capture exists for this workload, batch and GEMM source",
                    "flops_per_step": B * step_flops(shape)}
    if rank == 0:
        free_b, total_b = torch.cuda.mem_get_info()
        per_sample = L * planes * d * sbytes + 4 * w["gen"] + 4
        fixed = model.blob.numel() + ws.numel()
        max_conc = int((total_b * 0.97 - fixed) // per_sample)
        clocks = clk.summary(timed_regions)
        cpu = cpu_baseline(shape, W, args.workload, w) if world == 1 and not args.no_cpu_baseline else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": t_ms_max / args.steps, "higher_is_better": True,
            "blocks": {"n": len(block_ms), "steps_per_block": args.steps, "timed_s": round(sum(block_ms) / 1e3, 3),
                       "ms_per_step_median": round(t_ms_max / args.steps, 5),
                       "ms_per_step_min": round(min(block_ms) / args.steps, 5),
                       "ms_per_step_max": round(max(block_ms) / args.steps, 5),
                       "ms_per_step_first": round(block_ms[0] / args.steps, 5),
                       "note": "value and ms_per_step are the median block; every block is K steps between a "
                               "barrier + synchronize on both sides, MAX over ranks"},
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if shape.dtype == "bf16" else "f32",
            "data": "synthetic",
            "config": _config_dict(args, shape, w, B, extra={
                "state_dtype": args.state_dtype, "chunk_rows": chunk, "graph": args.graph, "ragged_prompts": bool(args.ragged),
                "l2": f"inputs larger than L2: per-step working set (cache {L * B * d * sbytes / 1e6:.0f} MB + weights "
                      f"{model.blob.numel() / 1e6:.0f} MB + logits {chunk * V * 4 / 1e6:.0f} MB) vs 126 MB L2; no flush"}),
            "gpu_launches": int(launches),
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": B * 4, "d2h_bytes_per_step": B * 4,
                    "ms_per_step": round(statistics.median(e2e_ms) / args.steps, 5), "blocks": len(e2e_ms),
                    "clocks": e2e_clocks},
            "roofline": roofline,
            "step_roofline": {"bound": bound, "t_roof_ms": round(t_roof * 1e3, 4), "t_tensor_ms": round(t_tc * 1e3, 4),
                              "t_hbm_ms": round(t_hbm * 1e3, 4), "frac": round(t_roof * 1e3 / (t_ms_max / args.steps), 4),
                              "peaks": f"{peak_src}: {peak_tf} TFLOP/s sustained bf16, {peaks['hbm_gbs']} GB/s HBM"},
            "kernels": kernels,
            "prefill": None if prefill_ms is None else
            {"ms": round(prefill_ms, 2), "prompt_tokens_per_s": round(B * n / (prefill_ms / 1e3), 1),
             "distinct_prompts": w.get("n_prompts") if (w["prompts"] == "replicated" and not args.no_prompt_dedup) else B},
            "state_bytes_per_sample": L * planes * d * sbytes,
            "max_concurrent_samples": max_conc,
            "device_status": status,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_sweep(args):
    """tokens/s vs batch on the mid model plus the largest batch that fits (128-token prompts,
    256 generated tokens per sample budgeted in the token store)."""
    import torch
    import paper_2605_08696_b200 as P
    import srm_inputs as I
    w = I.WORKLOADS["sweep"]
    shape = I.CONFIGS[w["model"]]
    dev = "cuda:0"
    torch.cuda.set_device(0)
    W = I.make_weights(shape)
    model = P.SRM(shape, W, device=dev, state_dtype=args.state_dtype)
    g = P.Sampling("greedy")
    sbytes = 4 if args.state_dtype == "fp32" else 2
    L, d = shape.n_layers, shape.d_model
    chunk = args.chunk
    ws = model.new_workspace(chunk, w["prompt_len"], prefill_samples=max(1, args.prefill_rows // w["prompt_len"]))
    free_b, total_b = torch.cuda.mem_get_info()
    per_sample = L * d * sbytes + 4 * w["gen"] + 4 + 4 * w["prompt_len"]
    max_conc = int((free_b * 0.97) // per_sample)
    batches = [1, 64, 1024, 8192, 32768]
    while batches[-1] * 2 <= max_conc:
        batches.append(batches[-1] * 2)
    if args.sweep_max:
        batches = [b for b in batches if b <= args.sweep_max]
    curve = []
    try:
        uuid = str(torch.cuda.get_device_properties(0).uuid)
    except Exception:
        uuid = None
    with ClockSampler(0, uuid) as clk:
        for B in batches:
            st = model.new_state(B)
            prompts = torch.from_numpy(I.uniform_prompts(min(B, 65536), w["prompt_len"], shape.vocab, shape.seed)).to(dev)
            if B > prompts.shape[0]:
                prompts = prompts.repeat((B + prompts.shape[0] - 1) // prompts.shape[0], 1)[:B].contiguous()
            model.prefill(st, prompts, g, ws)
            steps = 8 if B >= 262144 else 24
            store = torch.empty(B, steps, dtype=torch.int32, device=dev)
            model.generate(st, 4, 1, g, ws, out=store)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            # blocks of `steps` steps until MIN_TIMED_S has been timed (the context has room for 896 steps)
            blocks, n_target, region0 = [], None, len(clk.regions)
            while n_target is None or len(blocks) < n_target:
                if st.pos + steps > shape.n_ctx:
                    st.pos = w["prompt_len"]             # timing only: alpha/beta indices stay in range
                torch.cuda.synchronize()
                clk.mark_start()
                e0.record()
                model.generate(st, steps, 5, g, ws, out=store)
                e1.record()
                torch.cuda.synchronize()
                clk.mark_stop()
                blocks.append(e0.elapsed_time(e1))
                if n_target is None:
                    n_target = max(1, min(args.max_blocks, math.ceil(args.min_time * 1e3 / blocks[0])))
            ms = statistics.median(blocks) / steps
            curve.append({"batch": B, "ms_per_step": round(ms, 4), "tokens_per_s": round(B / (ms / 1e3), 1),
                          "blocks": len(blocks), "steps_per_block": steps,
                          "ms_per_step_min": round(min(blocks) / steps, 4), "ms_per_step_max": round(max(blocks) / steps, 4),
                          "state_bytes_per_sample": L * d * sbytes, "status": st.status(),
                          "clocks": clk.summary(clk.regions[region0:])})
            print(json.dumps(curve[-1]), file=sys.stderr, flush=True)
            del st, prompts, store
            torch.cuda.empty_cache()
    line = {"metric": METRIC, "unit": UNIT, "n_gpus": 1, "sweep": curve, "max_concurrent_samples": max_conc,
            "state_dtype": args.state_dtype, "config": {"workload": "sweep: mid SRM, 128-token uniform prompts"}}
    print(json.dumps(line), flush=True)


def run_variants(args):
    """Device time of the recurrent step of the two further mixer variants (linearly combined heads; kernels of
    size k, Eq. 11) on 65536 rows of d = 1024, against the bytes the step has to move. One JSON line."""
    import torch
    import paper_2605_08696_b200 as P
    dev = "cuda:0"
    torch.cuda.set_device(0)
    peaks, peak_src = measured_peaks()
    R, d, h, n_ctx = 65536, 1024, 4, 16
    gen = torch.Generator(device=dev).manual_seed(0)
    rnd = lambda *s: torch.randn(*s, device=dev, generator=gen)
    uni = lambda *s: torch.rand(*s, device=dev, generator=gen)

    def timed(f, n=20):
        for _ in range(3):
            f()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(n):
            f()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    z, y, beta = rnd(R, d), torch.empty(R, d, device=dev), rnd(n_ctx, d)
    S_r, S_c = rnd(R, d), rnd(R, d)
    a, lam, w = uni(h, n_ctx), uni(h) * 0.5, uni(h, 2)
    out = []
    ms = timed(lambda: P.k_mixer_combined_step(3, z, S_r, S_c, a, a, beta, lam, lam, w, y))
    out.append({"kernel": "combined_step_kernel", "rows": R, "d": d, "us": round(ms * 1e3, 1),
                "gbs": round(R * d * 24 / ms / 1e6, 1)})
    for k in (4, 8):
        Pk, al, lk = rnd(k, R, d), uni(k, n_ctx), uni(k) * 0.5
        ms = timed(lambda: P.k_mixer_kernel_step(3, z, Pk, al, beta, lk, y))
        out.append({"kernel": "kernel_mix_step_kernel", "k": k, "rows": R, "d": d, "us": round(ms * 1e3, 1),
                    "gbs": round(R * d * 4 * (2 * k + 2) / ms / 1e6, 1)})
    del S_r, S_c
    # the sequence form: 1024 prompts of 256 positions (8 bytes per element: input read, output written)
    Bp, n = 1024, 256
    Z, Y = rnd(Bp, n, d), torch.empty(Bp, n, d, device=dev)
    an, betan = uni(h, n), rnd(n, d)
    S_r, S_c = torch.zeros(Bp, d, device=dev), torch.zeros(Bp, d, device=dev)
    ms = timed(lambda: P.k_mixer_combined_scan(0, Z, S_r, S_c, an, an, betan, lam, lam, w, Y), n=10)
    out.append({"kernel": "combined_scan_kernel", "prompts": Bp, "n": n, "d": d, "us": round(ms * 1e3, 1),
                "gbs": round(Bp * n * d * 8 / ms / 1e6, 1)})
    for k in (4, 8):
        Pk, al, lk = torch.zeros(k, Bp, d, device=dev), uni(k, n), uni(k) * 0.5
        ms = timed(lambda: P.k_mixer_kernel_scan(0, Z, Pk, al, betan, lk, Y), n=10)
        out.append({"kernel": "kernel_scan_kernel", "k": k, "prompts": Bp, "n": n, "d": d, "us": round(ms * 1e3, 1),
                    "gbs": round(Bp * n * d * 8 / ms / 1e6, 1)})
    for o in out:
        o["frac_of_hbm_peak"] = round(o["gbs"] / peaks["hbm_gbs"], 3)
    print(json.dumps({"variants": out, "peak": f"{peak_src}: {peaks['hbm_gbs']} GB/s", "inputs": "larger than L2"}), flush=True)


def self_launch(n: int, argv) -> int:
    """`python bench.py --gpus N` without a launcher: start N local ranks (one process per GPU) of this same
    command through torch.distributed.run on the loopback address and return its exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mid", choices=["tiny", "small", "mid", "rl"])
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch per GPU")
    ap.add_argument("--chunk", type=int, default=8192, help="samples per decode pass (workspace size)")
    ap.add_argument("--prefill-rows", type=int, default=524288, help="prompt rows per prefill pass")
    ap.add_argument("--state-dtype", default="fp32", choices=["fp32", "fp16", "bf16"])
    ap.add_argument("--ref-samples", type=int, default=32)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--head-proj", action="store_true",
                    help="token mixer with head projections (Eq. 10): adds W_in, W_out [d, d] per layer")
    ap.add_argument("--mixer", default="mixed", choices=["mixed", "combined", "kernel"],
                    help="token mixer of the model: mixed heads (the hot path), linearly combined heads (twice the cache) "
                         "or kernels of size --kernel-size (Eq. 11; that many times the cache)")
    ap.add_argument("--kernel-size", type=int, default=4)
    ap.add_argument("--no-small-batch", action="store_true",
                    help="batches of at most 64 samples: one kernel per operation instead of the single-kernel step")
    ap.add_argument("--no-kslice", action="store_true",
                    help="small passes: down projection as whole tiles (no ranges of K with partial products)")
    ap.add_argument("--no-fused-ffn", action="store_true",
                    help="feed-forward block as two launches (up projection, down projection) instead of one kernel")
    ap.add_argument("--no-tail-split", action="store_true",
                    help="tensor-core projections keep the tiles of a partly filled last round whole (256 x 256)")
    ap.add_argument("--no-splitk", action="store_true",
                    help="down projection with whole output tiles per CTA pair (no sharing of K between pairs)")
    ap.add_argument("--ragged", action="store_true",
                    help="prompt lengths uniform on [n/2, n] (srm_prefill_ragged; one position per sample in the decode steps)")
    ap.add_argument("--top-p", type=float, default=None,
                    help="select tokens by nucleus sampling with this p (temperature 0.7 unless --temperature)")
    ap.add_argument("--temperature", type=float, default=None)
    ap.add_argument("--graph", default="auto", choices=["auto", "on", "off"],
                    help="srm_generate replays a captured step: auto = only for launch-bound (small) batches")
    ap.add_argument("--no-prompt-dedup", action="store_true",
                    help="rl workload: prefill all 16384 rows instead of the 16 distinct prompts")
    ap.add_argument("--no-prefill", action="store_true",
                    help="skip the prefill (cache stays zero, pos = prompt length): keeps profiler captures short")
    ap.add_argument("--min-time", type=float, default=MIN_TIMED_S,
                    help="the K-step block is repeated until this many seconds of device time have been timed")
    ap.add_argument("--max-blocks", type=int, default=400)
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--sweep-max", type=int, default=0)
    ap.add_argument("--variants", action="store_true",
                    help="time the stand-alone steps of the combined-head and kernel-size-k mixers")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(self_launch(args.gpus, sys.argv[1:]))
    elif args.sweep:
        run_sweep(args)
    elif args.variants:
        run_variants(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
