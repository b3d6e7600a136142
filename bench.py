#!/usr/bin/env python
"""Benchmark of the C2T draft-tree hot path.

A step is one decode step of the whole path over one batch of synthetic logits:
begin_step, D x (expand_level + prune), the Top-N rerank, the verification inputs and the
acceptance walk.  The workload at one GPU is B=64 sequences, V=128256, bf16 logits, D=8,
K=F=10, budget 60, threshold 0.5 (640 logits rows of 256 512 bytes per full level).

    python bench.py [--gpus N] [--steps K] [--warmup W]           the CUDA library
    python bench.py --impl reference [--steps K] [--warmup W]      the CPU oracle on a bounded sample

For N > 1 launch through torch.distributed.run: every rank owns its own B sequences (weak
scaling, no collective on the data path).  Rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time
from concurrent.futures import ThreadPoolExecutor

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import c2t_inputs  # noqa: E402

METRIC = "draft-tree levels/sec and µs per decode step; logits HBM GB/s vs ~8 TB/s"
UNIT = "levels/s"

WORKLOAD = dict(B=64, V=128256, D=8, K=10, F=10, N=60, beta=0.5, hidden=16)
REPEAT_BLOCKS = 6             # further blocks of `steps` steps after the headline block, for median / min / max
WORKLOAD_NAME = ("B=64 sequences, V=128256, bf16 draft and target logits, depth 8, top-k 10, frontier cap 10, "
                 "budget 60, threshold 0.5, MLP hidden 16")
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (read + write) of one expand_pass_kernel launch at this workload, from the ncu capture summarised in
# profiles/expand_pass_kernel_bf16_B64_V128256.txt: the 64-row launch of level 0 and a 640-row launch.  The counters
# belong to the kernel sources whose hash stands beside them: when a source changes the hash no longer matches and
# the bench reports no traffic figure until the counters (and the hash) are taken again.
EXPAND_DRAM_BYTES = {"level0": 16.49e6, "full_level": 167.77e6}
EXPAND_SOURCES = ("expand_pass.cu", "c2t_internal.h", "vocab_common.cuh")
EXPAND_SOURCES_SHA16 = "15c0e36ac9f6ade2"


def expand_dram_bytes():
    """The ncu counters above, or None if the kernel's sources are not the ones they were taken on."""
    h = hashlib.sha256()
    try:
        for name in EXPAND_SOURCES:
            with open(os.path.join(ROOT, "paper_2502_13652_b200", "csrc", name), "rb") as f:
                h.update(f.read())
    except OSError:
        return None
    return EXPAND_DRAM_BYTES if h.hexdigest()[:16] == EXPAND_SOURCES_SHA16 else None


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled every 20 ms in a child process."""
    FIELDS = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(gpu_index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        rows = []
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 10:
                continue
            try:
                ts = time.mktime(time.strptime(parts[0].split(".")[0], "%Y/%m/%d %H:%M:%S"))
                ts += float("0." + parts[0].split(".")[1]) if "." in parts[0] else 0.0
                rows.append((ts, float(parts[2]), float(parts[3]), parts[6:10]))
            except ValueError:
                continue
        self.file.close()
        os.unlink(self.file.name)
        inside = [r for r in rows if t0 - 0.05 <= r[0] <= t1 + 0.05]
        used = inside or rows[-3:]
        if not used:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm = sorted(r[1] for r in used)
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        reasons = sorted({n for r in used for n, v in zip(names, r[3]) if v.lower().startswith("active")})
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": used[0][2], "reasons": reasons,
                "samples": len(inside)}


# ---------------------------------------------------------------------------- sharding (host logic)

def rank_sequence_base(rank: int, batch_per_rank: int) -> int:
    """First global sequence id of a rank: ranks own disjoint blocks of `batch_per_rank` sequences."""
    return rank * batch_per_rank


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The slowest rank's figure (all-reduce MAX); the identity without a process group."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_levels_per_second(world: int, batch_per_rank: int, depth: int, ms_per_step: float) -> float:
    """Sequence-levels per second of the whole job: every rank advances its own sequences (weak scaling)."""
    return world * batch_per_rank * depth / (ms_per_step * 1e-3)


def make_weights(hidden):
    return c2t_inputs.classifier_weights(hidden, seed=0)


# ---------------------------------------------------------------------------- oracle arm

def oracle_sample(n_seq: int, step: int = 0, seq_base: int = 0):
    """Inputs of `n_seq` sequences of the workload on the CPU."""
    w = WORKLOAD
    draft = torch.stack([c2t_inputs.draft_logits(n_seq, w["F"], w["V"], step, l, torch.bfloat16, seq_base=seq_base)
                         for l in range(w["D"])], dim=1).contiguous()          # [n, D, F, V]
    target = c2t_inputs.target_logits(n_seq, w["N"], w["V"], step, torch.bfloat16, seq_base=seq_base)
    root = c2t_inputs.root_tokens(n_seq, w["V"], step, seq_base)
    prefix = c2t_inputs.prefix_lengths(n_seq, seq_base=seq_base)
    return draft, target, root, prefix


def oracle_config():
    import oracle
    w = WORKLOAD
    w1, b1, w2, b2 = make_weights(w["hidden"])
    return oracle.OracleConfig(vocab=w["V"], dtype=oracle.BF16, max_depth=w["D"], topk=w["K"],
                               frontier_cap=w["F"], budget=w["N"], threshold=w["beta"], hidden=w["hidden"],
                               w1=w1, b1=b1, w2=w2, b2=b2)


def host_cores() -> int:
    """Cores this process may run on."""
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def time_oracle(n_seq: int, steps: int, warmup: int, threads: int = 1):
    """Seconds per step of the oracle, as it stands, on n_seq sequences of the workload: one thread, or `threads`
    threads that each take whole sequences (the oracle works one sequence at a time and keeps no global state;
    the calls run outside the interpreter lock).  Returns (seconds per step, logits rows per step)."""
    import oracle
    oracle.build()
    draft, target, root, prefix = oracle_sample(n_seq)
    root, prefix = root.numpy(), prefix.numpy()
    for _ in range(warmup):
        oracle.decode_step(oracle_config(), draft[:1], target[:1], root[:1], prefix[:1])

    def one(b):
        return oracle.decode_step(oracle_config(), draft[b:b + 1], target[b:b + 1], root[b:b + 1],
                                  prefix[b:b + 1]).rows_visited

    t0 = time.perf_counter()
    rows = 0
    for _ in range(steps):
        if threads <= 1:
            rows += oracle.decode_step(oracle_config(), draft, target, root, prefix).rows_visited
        else:
            with ThreadPoolExecutor(max_workers=threads) as pool:
                rows += sum(pool.map(one, range(n_seq)))
    dt = (time.perf_counter() - t0) / steps
    return dt, rows // max(steps, 1)


MAX_ORACLE_THREADS = 16      # bounds the sample (one sequence per thread) and the time spent generating it


def oracle_baseline(steps: int, warmup: int):
    """The oracle on this host: threads over sequences on the cores this process may use (at most
    MAX_ORACLE_THREADS), and on one core.  Returns the `cpu_baseline` object of the JSON line and ms per step."""
    w = WORKLOAD
    cores = host_cores()
    threads = min(cores, MAX_ORACLE_THREADS)
    n_seq = max(threads, 2)
    dt, rows = time_oracle(n_seq, steps, warmup, threads)
    value = n_seq * w["D"] / dt
    n1 = 2
    dt1, rows1 = time_oracle(n1, 1, 0, 1)
    sample = (f"{n_seq} of the workload's {w['B']} sequences per step, one sequence per thread (all {w['D']} levels, "
              f"rerank, verify inputs, accept walk; {rows} logits rows of {w['V']} bf16 per step), {dt:.1f} s per step")
    return {"value": value, "unit": UNIT, "cores": threads, "host_cores": cores, "kind": "oracle", "sample": sample,
            "single_core": {"value": n1 * w["D"] / dt1, "unit": UNIT, "cores": 1,
                            "sample": f"{n1} sequences, one step ({rows1} logits rows), {dt1:.1f} s"}}, dt * 1e3


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    base, ms = oracle_baseline(args.steps, min(args.warmup, 1))
    line = {
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAME, "sample": base["sample"]},
        "cpu_baseline": base,
        "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "us_per_step": ms * 1e3,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------- CUDA arm

def run_cuda(args) -> None:
    import paper_2502_13652_b200 as c2t

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA arm has no CPU fallback")
    if not os.path.exists(c2t.LIB_PATH):
        from paper_2502_13652_b200 import build
        build.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    w = WORKLOAD
    B, V, D, K, F, N = w["B"], w["V"], w["D"], w["K"], w["F"], w["N"]
    w1, b1, w2, b2 = make_weights(w["hidden"])
    cfg = c2t.Config(batch=B, vocab=V, dtype=c2t.BF16, max_depth=D, topk=K, frontier_cap=F, budget=N,
                     threshold=w["beta"], hidden=w["hidden"], w1=w1, b1=b1, w2=w2, b2=b2, device=local_rank)
    ctx = c2t.Context(cfg)
    Nw = ctx.Nw
    seq_base = rank_sequence_base(rank, B)                # every rank owns its own sequences
    draft = [c2t_inputs.draft_logits(B, F, V, 0, l, torch.bfloat16, device=dev, seq_base=seq_base)
             for l in range(D)]
    target = c2t_inputs.target_logits(B, Nw, V, 0, torch.bfloat16, device=dev, seq_base=seq_base)
    root = c2t_inputs.root_tokens(B, V, 0, seq_base).to(dev)
    prefix = c2t_inputs.prefix_lengths(B, seq_base=seq_base).to(dev)
    default_stream = stream = torch.cuda.current_stream().cuda_stream

    def step(events=None, lazy=False, stream_handle=None, target=target):
        stream = stream_handle if stream_handle is not None else default_stream
        ctx.c2t_begin_step(root, prefix, stream)
        for l in range(D):
            if events is not None:
                events[2 * l].record()
            ctx.c2t_expand_level(l, draft[l], stream)
            if events is not None:
                events[2 * l + 1].record()
            ctx.c2t_prune(l, stream)
        ctx.c2t_prune(c2t.FINAL, stream)
        ctx.c2t_build_verify(stream)
        if lazy:
            ctx.c2t_accept_lazy(target, stream)
        else:
            ctx.c2t_accept(target, stream)

    # active rows per level (the same every step: the inputs do not change)
    ctx.c2t_begin_step(root, prefix, stream)
    rows_per_level = []
    for l in range(D):
        rows_per_level.append(int(ctx.c2t_get_view()["frontier_n"].sum().item()))
        ctx.c2t_expand_level(l, draft[l], stream)
        ctx.c2t_prune(l, stream)
    ctx.c2t_prune(c2t.FINAL, stream)
    ctx.c2t_build_verify(stream)
    ctx.c2t_accept(target, stream)
    torch.cuda.synchronize()
    status, _ = ctx.c2t_status()
    n_nodes = ctx.verify["n_nodes"].cpu()
    accept_len = ctx.accepted["accept_len"].cpu()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    time.sleep(0.15 if sampler else 0.0)
    # events around the expand launches of every 8th step only: recording 16 events in every step costs 7 % of it
    sampled = [s for s in range(args.steps) if s % 8 == 0]
    evs = {s: [torch.cuda.Event(enable_timing=True) for _ in range(2 * D)] for s in sampled}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.c2t_launch_count()
    barrier()
    t_wall0 = time.time()
    e0.record()
    for s in range(args.steps):
        step(evs.get(s))
    e1.record()
    barrier()
    t_wall1 = time.time()
    launches = ctx.c2t_launch_count() - launches0
    ms_total = e0.elapsed_time(e1)
    expand_ms = sum(evs[s][2 * l].elapsed_time(evs[s][2 * l + 1]) for s in sampled for l in range(D))
    full_ms = [evs[s][2 * l].elapsed_time(evs[s][2 * l + 1]) for s in sampled for l in range(1, D)]

    ms_total_max = max_over_ranks(ms_total, dist, dev)
    ms_per_step = ms_total_max / args.steps
    value = whole_job_levels_per_second(world, B, D, ms_per_step)

    # ---- the same block of `steps` steps a few more times: median and range beside the headline (which is the
    # first block, as timed above); the clock samples cover these blocks too
    block_ms = [ms_per_step]
    for _ in range(REPEAT_BLOCKS):
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        r0.record()
        for s in range(args.steps):
            step()
        r1.record()
        barrier()
        block_ms.append(max_over_ranks(r0.elapsed_time(r1), dist, dev) / args.steps)
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None

    # ---- the same steps with the acceptance walk that reads only the rows it visits (reported beside the
    # headline, which keeps the all-rows arg-max of the workload definition)
    for _ in range(3):
        step(lazy=True)
    barrier()
    z0, z1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    z0.record()
    for s in range(args.steps):
        step(lazy=True)
    z1.record()
    barrier()
    lazy_ms_per_step = max_over_ranks(z0.elapsed_time(z1), dist, dev) / args.steps
    assert torch.equal(ctx.accepted["accept_len"].cpu(), accept_len)

    # ---- both acceptance calls on target rows whose arg-maxes follow a path of the final tree (2 to 5 levels
    # deep, 3.5 on average where the trees allow it): the synthetic target rows alone accept almost nothing, so
    # the walk never moves and the lazy call reads one row per sequence; with planted paths it reads tau + 1
    target_planted, planted_depth = plant_accept_paths(ctx, target, V)
    planted = {}
    for name, lazy in (("all_rows", False), ("lazy", True)):
        for _ in range(3):
            step(lazy=lazy, target=target_planted)
        barrier()
        y0, y1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        y0.record()
        for s in range(args.steps):
            step(lazy=lazy, target=target_planted)
        y1.record()
        barrier()
        planted[name] = max_over_ranks(y0.elapsed_time(y1), dist, dev) / args.steps
        assert ctx.accepted["accept_len"].cpu().tolist() == planted_depth
    del target_planted

    # ---- the same step captured once in a CUDA graph and replayed (all-rows accept): what a serving loop
    # without a draft model between the levels would do; reported beside the headline
    graph_ms_per_step = None
    try:
        side = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(side):
            step(stream_handle=side.cuda_stream)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step(stream_handle=torch.cuda.current_stream().cuda_stream)
        for _ in range(3):
            graph.replay()
        barrier()
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        q0.record()
        for _ in range(args.steps):
            graph.replay()
        q1.record()
        barrier()
        graph_ms_per_step = max_over_ranks(q0.elapsed_time(q1), dist, dev) / args.steps
        assert torch.equal(ctx.accepted["accept_len"].cpu(), accept_len)
    except RuntimeError as exc:                      # capture not possible here: the figure is simply absent
        print(f"bench.py: CUDA graph replay skipped: {exc}", file=sys.stderr)

    # ---- end to end through the host-buffer entry point (pinned host logits in, results out)
    e2e_steps = max(1, min(args.steps, 5))
    stage, results = ctx.host_step_buffers()
    draft_host = [t_.cpu().pin_memory() for t_ in draft]
    target_host = target.cpu().pin_memory()
    root_host, prefix_host = root.cpu().pin_memory(), prefix.cpu().pin_memory()
    ctx.c2t_decode_step_host(draft_host, target_host, root_host, prefix_host, results, stage, stream)
    barrier()
    t0 = time.perf_counter()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for _ in range(e2e_steps):
        ctx.c2t_decode_step_host(draft_host, target_host, root_host, prefix_host, results, stage, stream)
    g1.record()
    barrier()
    e2e_ms = max(g0.elapsed_time(g1), (time.perf_counter() - t0) * 1e3) / e2e_steps
    e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    assert torch.equal(results["accept_len"], accept_len) and torch.equal(results["n_nodes"], n_nodes)
    eb = 2
    h2d = B * V * eb + (D - 1) * B * F * V * eb + B * Nw * V * eb + 2 * B * 4
    d2h = 4 * (B + B * Nw + B + B * (D + 1) + B)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- the same expand kernel on fp32 logits (twice the bytes per element, the same arithmetic per element):
    # reported beside the bf16 figure to show which side of the kernel the bytes-per-element ratio puts the bound on
    fp32_level = expand_full_level(c2t, dev, (w1, b1, w2, b2), root, prefix, default_stream, torch.float32, 4.0)
    # ... and on flat logits (temperature scale 1), where the kernel's work per element is at its largest
    scale1_level = expand_full_level(c2t, dev, (w1, b1, w2, b2), root, prefix, default_stream, torch.bfloat16, 1.0)
    topm_level = expand_full_level(c2t, dev, (w1, b1, w2, b2), root, prefix, default_stream, torch.bfloat16, 4.0,
                                   top_m=1000)

    # ---- the single-sequence configuration (latency-bound), timed per decode step; one GPU only
    single_seq = single_sequence_latency(c2t, dev, default_stream) if world == 1 else None
    configs = None
    if world == 1:
        configs = {"config1": config1_single_sequence_fp32(c2t, dev, default_stream),
                   "config2": config2_chained_steps(c2t, dev, default_stream),
                   "config3": "single_sequence (below)",
                   "config5": config5_ablation_sweep(c2t, dev, default_stream)}

    # ---- roofline of the dominant kernel (the per-level vocabulary pass)
    peak, peak_kind = measured_hbm_peak()
    bytes_per_launch = sum(rows_per_level) * V * eb / D
    avg_launch_s = expand_ms * 1e-3 / (len(sampled) * D)
    achieved = bytes_per_launch / avg_launch_s / 1e9
    full_rows = max(rows_per_level[1:]) if D > 1 else rows_per_level[0]
    full_level_gbs = None
    if full_ms:
        full_bytes = sum(rows_per_level[1:]) * V * eb / (D - 1)
        full_level_gbs = full_bytes / (sum(full_ms) / len(full_ms) * 1e-3) / 1e9

    # DRAM bytes per launch (ncu: dram__bytes_read.sum + dram__bytes_write.sum of this kernel at this workload's
    # two launch shapes, profiles/expand_pass_kernel_bf16_B64_V128256.txt), scaled by the rows a launch streams
    # and averaged over the step's launches like `achieved`.  None when the counters do not cover the workload.
    traffic = None
    dram = expand_dram_bytes()
    if (B, V, F) == (64, 128256, 10) and dram is not None:
        per_row = [dram["level0"] / 64.0] + [dram["full_level"] / 640.0] * (D - 1)
        traffic = sum(r * b for r, b in zip(rows_per_level, per_row)) / D

    # ---- the oracle on this host, bounded sample
    cpu_base, _ = oracle_baseline(1, 1)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAME, "value_counts": "sequence-levels per second (B*D per step, all ranks)",
                   "l2": "inputs larger than L2: 1.17 GB of draft rows and 0.98 GB of target rows per step",
                   "rows_per_level": rows_per_level, "mean_final_nodes": float(n_nodes.float().mean()),
                   "mean_accept_len": float(accept_len.float().mean()), "status_bits": status,
                   "parallelism": f"dp{world} (independent sequences per rank, no collective)"},
        "us_per_step": ms_per_step * 1e3, "us_per_level": ms_per_step * 1e3 / D,
        "us_per_step_blocks": {"n": len(block_ms), "steps_per_block": args.steps,
                               "median": statistics.median(block_ms) * 1e3, "min": min(block_ms) * 1e3,
                               "max": max(block_ms) * 1e3},
        "graph_replay": None if graph_ms_per_step is None else {
            "us_per_step": graph_ms_per_step * 1e3,
            "value": whole_job_levels_per_second(world, B, D, graph_ms_per_step), "unit": UNIT,
            "note": "the step's 21 launches captured once in a CUDA graph and replayed"},
        "lazy_accept": {"us_per_step": lazy_ms_per_step * 1e3,
                        "value": whole_job_levels_per_second(world, B, D, lazy_ms_per_step), "unit": UNIT,
                        "mean_accept_len": float(accept_len.float().mean()),
                        "note": "c2t_accept_lazy: accept_len+1 target rows per sequence instead of all final nodes",
                        "planted_paths": {
                            "mean_accept_len": sum(planted_depth) / len(planted_depth),
                            "target_rows_read_per_sequence": sum(planted_depth) / len(planted_depth) + 1,
                            "us_per_step_lazy": planted["lazy"] * 1e3,
                            "us_per_step_all_rows": planted["all_rows"] * 1e3,
                            "note": "target arg-maxes planted along a path of each final tree"}},
        "single_sequence": single_seq,
        "configs": configs,
        "clocks": clocks,
        "e2e": {"value": whole_job_levels_per_second(world, B, D, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "expand_pass_kernel<bf16>", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "traffic": traffic, "traffic_unit": "DRAM bytes per launch (ncu, read + write)",
                     "bytes_per_launch": bytes_per_launch,
                     "avg_launch_us": avg_launch_s * 1e6,
                     "full_level_rows": full_rows, "full_level_gbs": full_level_gbs,
                     "frac_of_8000": achieved / 8000.0,
                     "us_x_sm_mhz": None if not clocks or not clocks.get("sm_mhz") else
                     avg_launch_s * 1e6 * clocks["sm_mhz"],
                     "fp32_logits_full_level": None if fp32_level is None else dict(
                         fp32_level, frac=fp32_level["gbs"] / peak),
                     "scale1_logits_full_level": None if scale1_level is None else dict(
                         scale1_level, frac=scale1_level["gbs"] / peak, frac_of_8000=scale1_level["gbs"] / 8000.0),
                     "truncated_entropy_full_level": topm_level},
        "cpu_baseline": cpu_base,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def plant_accept_paths(ctx, target, V, depths=(2, 3, 4, 5)):
    """A copy of `target` in which, per sequence, the arg-maxes of the rows along one root-to-leaf path of the final
    tree (as the context's last step left it) point to the next node of the path, down to a chosen depth, and the
    row at that depth points to a token none of its children carries.  Returns (tensor, accept length per sequence)."""
    ver = {k: v.cpu().numpy() for k, v in ctx.verify.items()}
    out = target.clone()
    got = []
    for b in range(ctx.B):
        n = int(ver["n_nodes"][b])
        rows = ver["retrieve"][b, :int(ver["n_leaves"][b])]
        chain = max(([int(x) for x in r if x >= 0] for r in rows), key=len)     # the deepest path
        d = min(depths[b % len(depths)], len(chain) - 1)
        for here, nxt in zip(chain[:d], chain[1:d + 1]):
            out[b, here, int(ver["tokens"][b, nxt])] = 1000.0
        kids = {int(ver["tokens"][b, i]) for i in range(n) if int(ver["parents"][b, i]) == chain[d]}
        out[b, chain[d], next(t for t in range(V) if t not in kids)] = 1000.0
        got.append(d)
    return out, got


def expand_full_level(c2t, dev, weights, root, prefix, stream, dtype=torch.float32, scale: float = 4.0,
                      reps: int = 20, top_m: int = 0):
    """Times the expand kernel on full levels of the workload with other logits than the headline's: fp32 instead
    of bf16, or another temperature scale (levels 1-3, three distinct buffers, so every launch reads from DRAM).
    top_m > 0: with the truncated entropy of Eq. 3, whose kernels run inside the same call (the time is then that of
    the pass plus those).  Returns None if the frontier does not fill."""
    w = WORKLOAD
    B, V, K, F, N = w["B"], w["V"], w["K"], w["F"], w["N"]
    levels = 4
    w1, b1, w2, b2 = weights
    cfg = c2t.Config(batch=B, vocab=V, dtype=c2t.F32 if dtype == torch.float32 else c2t.BF16, max_depth=levels,
                     topk=K, frontier_cap=F, budget=N, threshold=0.0, classifier=c2t.CLS_IDENTITY_JOINT,
                     hidden=w["hidden"], w1=w1, b1=b1, w2=w2, b2=b2, device=dev.index, entropy_top_m=top_m)
    ctx = c2t.Context(cfg)
    draft = [c2t_inputs.draft_logits(B, F, V, 0, l, dtype, scale, device=dev) for l in range(levels)]
    rows = []
    ms = []
    from_pass = None
    for rep in range(reps + 3):
        ctx.c2t_begin_step(root, prefix, stream)
        for l in range(levels):
            if rep == 0:
                rows.append(int(ctx.c2t_get_view()["frontier_n"].sum().item()))
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            ctx.c2t_expand_level(l, draft[l], stream)
            b.record()
            if top_m and rep == 0 and l == 1:
                from_pass = int(ctx.c2t_get_view()["topm_from_pass"].sum().item())
            ctx.c2t_prune(l, stream)
            if rep >= 3 and l >= 1:
                ms.append((a, b))
    torch.cuda.synchronize()
    if min(rows[1:]) != B * F:
        return None
    t = sorted(a.elapsed_time(b) * 1e3 for a, b in ms)
    us = sum(t) / len(t)
    nbytes = B * F * V * (4 if dtype == torch.float32 else 2)
    ctx.close()
    out = {"rows": B * F, "bytes": nbytes, "us": us, "us_median": t[len(t) // 2], "us_min": t[0],
           "gbs": nbytes / (us * 1e-6) / 1e9, "scale": scale, "dtype": "f32" if dtype == torch.float32 else "bf16",
           "note": "threshold 0 with the identity classifier, so that every level has B*F active rows"}
    if top_m:
        out["entropy_top_m"] = top_m
        out["rows_served_from_the_pass"] = from_pass
        out["note"] += "; the time covers the pass, the per-row selection and the (empty) second-read launch"
    return out


def single_sequence_latency(c2t, dev, stream, steps: int = 60, sets: int = 4):
    """The single-stream case: B=1, V=128256, bf16, D=10, K=8, F=16, N=80, thresholds 0.3 / 0.5 / 0.7; µs per decode
    step.  One step's logits (61 MB) would stay in L2, so the steps rotate over `sets` input sets (246 MB)."""
    B, V, D, K, F, N, hidden = 1, 128256, 10, 8, 16, 80, 16
    w1, b1, w2, b2 = make_weights(hidden)
    out = {"workload": "B=1, V=128256, bf16, depth 10, top-k 8, frontier cap 16, budget 80, MLP hidden 16",
           "l2": f"steps rotate over {sets} input sets (246 MB, larger than L2)", "us_per_step": {}, "us_per_step_graph_replay": {}, "rows_per_step": {}}
    inputs = None
    for beta in (0.3, 0.5, 0.7):
        cfg = c2t.Config(batch=B, vocab=V, dtype=c2t.BF16, max_depth=D, topk=K, frontier_cap=F, budget=N,
                         threshold=beta, hidden=hidden, w1=w1, b1=b1, w2=w2, b2=b2, device=dev.index)
        ctx = c2t.Context(cfg)
        if inputs is None:
            inputs = []
            for k in range(sets):
                draft = [c2t_inputs.draft_logits(B, F, V, k, l, torch.bfloat16, device=dev) for l in range(D)]
                target = c2t_inputs.target_logits(B, ctx.Nw, V, k, torch.bfloat16, device=dev)
                inputs.append((draft, target, c2t_inputs.root_tokens(B, V, k).to(dev),
                               c2t_inputs.prefix_lengths(B).to(dev)))
        rows = 0
        ctx.c2t_begin_step(inputs[0][2], inputs[0][3], stream)
        for l in range(D):
            rows += int(ctx.c2t_get_view()["frontier_n"].sum().item())
            ctx.c2t_expand_level(l, inputs[0][0][l], stream)
            ctx.c2t_prune(l, stream)
        for i in range(4):
            ctx.decode_step(*inputs[i % sets], stream=stream)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(steps):
            ctx.decode_step(*inputs[i % sets], stream=stream)
        b.record()
        torch.cuda.synchronize()
        out["us_per_step"][str(beta)] = a.elapsed_time(b) / steps * 1e3
        out["rows_per_step"][str(beta)] = rows
        # the same steps replayed from CUDA graphs (one per input set): 24 launches of a few microseconds each are
        # bounded by the host's launch calls otherwise
        try:
            side = torch.cuda.Stream(device=dev)
            graphs = []
            for k in range(sets):
                with torch.cuda.stream(side):
                    ctx.decode_step(*inputs[k], stream=side.cuda_stream)
                torch.cuda.synchronize()
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr, stream=side):
                    ctx.decode_step(*inputs[k], stream=torch.cuda.current_stream().cuda_stream)
                graphs.append(gr)
            for i in range(4):
                graphs[i % sets].replay()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(steps):
                graphs[i % sets].replay()
            b.record()
            torch.cuda.synchronize()
            out["us_per_step_graph_replay"][str(beta)] = a.elapsed_time(b) / steps * 1e3
            del graphs
        except RuntimeError as exc:
            print(f"bench.py: CUDA graph replay of the single-sequence case skipped: {exc}", file=sys.stderr)
        ctx.close()
    return out


def _time_steps(fn, n, warm=3):
    for i in range(warm):
        fn(i)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(n):
        fn(warm + i)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / n * 1e3


def config1_single_sequence_fp32(c2t, dev, stream, steps: int = 120, sets: int = 12):
    """B=1, V=32000, fp32, D=6, K=F=10, N=60, threshold 0.5: microseconds per decode step.  A step's logits (15 MB)
    would stay in L2, so the steps rotate over `sets` input sets (185 MB)."""
    B, V, D, K, F, N, hidden = 1, 32000, 6, 10, 10, 60, 16
    w1, b1, w2, b2 = make_weights(hidden)
    cfg = c2t.Config(batch=B, vocab=V, dtype=c2t.F32, max_depth=D, topk=K, frontier_cap=F, budget=N, threshold=0.5,
                     hidden=hidden, w1=w1, b1=b1, w2=w2, b2=b2, device=dev.index)
    ctx = c2t.Context(cfg)
    inputs = []
    for k in range(sets):
        inputs.append(([c2t_inputs.draft_logits(B, F, V, k, l, torch.float32, device=dev) for l in range(D)],
                       c2t_inputs.target_logits(B, ctx.Nw, V, k, torch.float32, device=dev),
                       c2t_inputs.root_tokens(B, V, k).to(dev), c2t_inputs.prefix_lengths(B).to(dev)))
    nodes, taus = [], []
    for k in range(sets):
        ctx.decode_step(*inputs[k], stream=stream)
        nodes.append(int(ctx.verify["n_nodes"][0])); taus.append(int(ctx.accepted["accept_len"][0]))
    us = _time_steps(lambda i: ctx.decode_step(*inputs[i % sets], stream=stream), steps)
    ctx.close()
    return {"workload": "B=1, V=32000, fp32, depth 6, top-k 10, frontier cap 10, budget 60, threshold 0.5, MLP hidden 16",
            "l2": f"steps rotate over {sets} input sets (185 MB, larger than L2)", "us_per_step": us,
            "mean_final_nodes": sum(nodes) / sets, "mean_accept_len": sum(taus) / sets}


def config2_chained_steps(c2t, dev, stream, steps: int = 64, sets: int = 16):
    """B=8, V=32000, bf16, D=8, K=F=10, N=60, threshold 0.5: 64 decode steps in a row, each starting from the
    previous step's next token and from a prefix that is accept_len + 1 tokens longer (the state stays on the
    device).  The logits of step s are input set s mod `sets` (16 sets, 1.2 GB)."""
    B, V, D, K, F, N, hidden = 8, 32000, 8, 10, 10, 60, 16
    w1, b1, w2, b2 = make_weights(hidden)
    cfg = c2t.Config(batch=B, vocab=V, dtype=c2t.BF16, max_depth=D, topk=K, frontier_cap=F, budget=N, threshold=0.5,
                     hidden=hidden, w1=w1, b1=b1, w2=w2, b2=b2, device=dev.index)
    ctx = c2t.Context(cfg)
    inputs = [([c2t_inputs.draft_logits(B, F, V, k, l, torch.bfloat16, device=dev) for l in range(D)],
               c2t_inputs.target_logits(B, ctx.Nw, V, k, torch.bfloat16, device=dev)) for k in range(sets)]
    root0 = c2t_inputs.root_tokens(B, V, 0).to(dev)
    prefix0 = c2t_inputs.prefix_lengths(B).to(dev)

    def chain(record):
        root, prefix = root0, prefix0
        for s in range(steps):
            ctx.decode_step(inputs[s % sets][0], inputs[s % sets][1], root, prefix, stream=stream)
            if record is not None:
                record.append((ctx.verify["n_nodes"].clone(), ctx.accepted["accept_len"].clone()))
            root = ctx.accepted["next_token"].clone()
            prefix = prefix + ctx.accepted["accept_len"] + 1
        return prefix

    rec = []
    chain(rec)                                          # warm-up, and the counts (the chain is deterministic)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    last_prefix = chain(None)
    b.record()
    torch.cuda.synchronize()
    nodes = torch.stack([r[0] for r in rec]).float()
    taus = torch.stack([r[1] for r in rec]).float()
    grown = (last_prefix - prefix0).float().mean().item()
    ctx.close()
    return {"workload": "B=8, V=32000, bf16, depth 8, top-k 10, frontier cap 10, budget 60, threshold 0.5, 64 chained steps",
            "us_per_step": a.elapsed_time(b) / steps * 1e3, "steps": steps, "mean_accept_len": taus.mean().item(),
            "mean_final_nodes": nodes.mean().item(), "mean_tokens_committed_per_sequence": grown}


def config5_ablation_sweep(c2t, dev, stream, depth: int = 8, steps: int = 8):
    """B=32; vocabulary {32000, 128256} x dtype {fp32, bf16} x temperature scale {1, 4, 8} x classifier {identity
    on the joint probability (EAGLE-2's expand + rerank), the FFN at threshold 0.5} x budget {20, 40, 60, 80} at
    depth 8: kept candidates, accept length against the synthetic target rows, microseconds per level."""
    B, K, F, hidden = 32, 10, 10, 16
    w1, b1, w2, b2 = make_weights(hidden)
    rows = []
    for V in (32000, 128256):
        for dtype in (torch.float32, torch.bfloat16):
            for scale in (1.0, 4.0, 8.0):
                draft = [c2t_inputs.draft_logits(B, F, V, 0, l, dtype, scale, device=dev) for l in range(depth)]
                target = c2t_inputs.target_logits(B, 80, V, 0, dtype, scale, device=dev)
                root = c2t_inputs.root_tokens(B, V, 0).to(dev)
                prefix = c2t_inputs.prefix_lengths(B).to(dev)
                for classifier, beta in ((c2t.CLS_IDENTITY_JOINT, 0.0), (c2t.CLS_MLP, 0.5)):
                    for N in (20, 40, 60, 80):
                        cfg = c2t.Config(batch=B, vocab=V, dtype=c2t.F32 if dtype == torch.float32 else c2t.BF16,
                                         max_depth=depth, topk=K, frontier_cap=F, budget=N, threshold=beta,
                                         classifier=classifier, hidden=hidden, w1=w1, b1=b1, w2=w2, b2=b2,
                                         device=dev.index)
                        ctx = c2t.Context(cfg)
                        us = _time_steps(lambda i: ctx.decode_step(draft, target, root, prefix, stream=stream), steps, 2)
                        view = ctx.c2t_get_view()
                        rows.append({"V": V, "dtype": "f32" if dtype == torch.float32 else "bf16", "scale": scale,
                                     "classifier": "identity_joint" if classifier == c2t.CLS_IDENTITY_JOINT else "mlp",
                                     "budget": N, "mean_tree_nodes_before_rerank": view["tree_n"].float().mean().item(),
                                     "mean_final_nodes": ctx.verify["n_nodes"].float().mean().item(),
                                     "mean_accept_len": ctx.accepted["accept_len"].float().mean().item(),
                                     "us_per_level": us / depth})      # whole step / depth
                        ctx.close()
                del draft, target
    return {"workload": f"B=32, depth {depth}, top-k 10, frontier cap 10; the same step repeated {steps} times "
                        "(logits of the larger cases exceed L2)", "rows": rows}


def run_profile(args) -> None:
    """Levels 0 and 1 of the workload (64 + 640 logits rows) and the tail of the step, `steps` times."""
    import paper_2502_13652_b200 as c2t
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = WORKLOAD
    B, V, D, K, F, N = w["B"], w["V"], w["D"], w["K"], w["F"], w["N"]
    w1, b1, w2, b2 = make_weights(w["hidden"])
    tdt = torch.float32 if args.profile_dtype == "f32" else torch.bfloat16
    cfg = c2t.Config(batch=B, vocab=V, dtype=c2t.F32 if tdt == torch.float32 else c2t.BF16, max_depth=D, topk=K,
                     frontier_cap=F, budget=N, threshold=w["beta"], hidden=w["hidden"], w1=w1, b1=b1, w2=w2, b2=b2,
                     entropy_top_m=args.profile_top_m)
    ctx = c2t.Context(cfg)
    draft = [c2t_inputs.draft_logits(B, F, V, 0, l, tdt, device=dev) for l in range(2)]
    target = c2t_inputs.target_logits(B, ctx.Nw, V, 0, tdt, device=dev)
    root = c2t_inputs.root_tokens(B, V, 0).to(dev)
    prefix = c2t_inputs.prefix_lengths(B).to(dev)
    for _ in range(args.warmup + args.steps):
        ctx.c2t_begin_step(root, prefix)
        for l in range(2):
            ctx.c2t_expand_level(l, draft[l])
            ctx.c2t_prune(l)
        ctx.c2t_prune(c2t.FINAL)
        ctx.c2t_build_verify()
        ctx.c2t_accept(target)
    torch.cuda.synchronize()
    print(json.dumps({"profile": True, "launches": ctx.c2t_launch_count(),
                      "n_nodes_mean": float(ctx.verify["n_nodes"].float().mean())}))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["cuda", "reference"], default="cuda")
    ap.add_argument("--profile", action="store_true",
                    help="small run for profiler captures: levels 0-1 of the workload plus rerank, verify "
                         "inputs and accept; no end-to-end leg, no CPU baseline")
    ap.add_argument("--profile-dtype", choices=["bf16", "f32"], default="bf16", help="logits dtype of the --profile run")
    ap.add_argument("--profile-top-m", type=int, default=0, help="entropy_top_m of the --profile run (Eq. 3)")
    args = ap.parse_args()
    if args.profile:
        args.steps = args.steps or 1
        run_profile(args)
        return
    if args.impl == "reference":
        args.steps = args.steps or 5
        run_reference(args)
    else:
        args.steps = args.steps or 1000
        run_cuda(args)


if __name__ == "__main__":
    main()
