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
import json
import os
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import c2t_inputs  # noqa: E402

METRIC = "draft-tree levels/sec and µs per decode step; logits HBM GB/s vs ~8 TB/s"
UNIT = "levels/s"

WORKLOAD = dict(B=64, V=128256, D=8, K=10, F=10, N=60, beta=0.5, hidden=16)
WORKLOAD_NAME = ("B=64 sequences, V=128256, bf16 draft and target logits, depth 8, top-k 10, frontier cap 10, "
                 "budget 60, threshold 0.5, MLP hidden 16")
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (read + write) of one expand_pass_kernel launch at this workload, from the ncu capture summarised in
# profiles/expand_pass_kernel_bf16_B64_V128256.txt: the 64-row launch of level 0 and a 640-row launch.  Set to
# None when the kernel changes until the counters are taken again.
EXPAND_DRAM_BYTES = {"level0": 16.49e6, "full_level": 168.09e6}


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled every 50 ms in a child process."""
    FIELDS = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
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


def time_oracle(n_seq: int, steps: int, warmup: int):
    """Seconds per step of the oracle on n_seq sequences (single thread)."""
    import oracle
    oracle.build()
    cfg = oracle_config()
    draft, target, root, prefix = oracle_sample(n_seq)
    for _ in range(warmup):
        oracle.decode_step(cfg, draft[:1], target[:1], root[:1].numpy(), prefix[:1].numpy())
    t0 = time.perf_counter()
    rows = 0
    for _ in range(steps):
        rows += oracle.decode_step(cfg, draft, target, root.numpy(), prefix.numpy()).rows_visited
    dt = (time.perf_counter() - t0) / steps
    return dt, rows // max(steps, 1)


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_seq = 2
    dt, rows = time_oracle(n_seq, args.steps, min(args.warmup, 1))
    value = n_seq * WORKLOAD["D"] / dt
    sample = (f"{n_seq} of the workload's 64 sequences per step (all {WORKLOAD['D']} levels, rerank, verify "
              f"inputs, accept walk; {rows} logits rows of {WORKLOAD['V']} bf16 per step)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAME, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "us_per_step": dt * 1e6,
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

    def step(events=None, lazy=False, stream_handle=None):
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
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None

    ms_total_max = max_over_ranks(ms_total, dist, dev)
    ms_per_step = ms_total_max / args.steps
    value = whole_job_levels_per_second(world, B, D, ms_per_step)

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
    fp32_level = expand_full_level_fp32(c2t, dev, (w1, b1, w2, b2), root, prefix, default_stream)

    # ---- the single-sequence configuration (latency-bound), timed per decode step; one GPU only
    single_seq = single_sequence_latency(c2t, dev, default_stream) if world == 1 else None

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
    if (B, V, F) == (64, 128256, 10) and EXPAND_DRAM_BYTES is not None:
        per_row = [EXPAND_DRAM_BYTES["level0"] / 64.0] + [EXPAND_DRAM_BYTES["full_level"] / 640.0] * (D - 1)
        traffic = sum(r * b for r, b in zip(rows_per_level, per_row)) / D

    # ---- the oracle on this host, bounded sample
    n_seq = 8
    dt_cpu, rows_cpu = time_oracle(n_seq, 1, 1)
    cpu_value = n_seq * D / dt_cpu
    sample = (f"{n_seq} of the workload's {B} sequences, one decode step ({rows_cpu} logits rows of {V} bf16), "
              f"{dt_cpu:.1f} s")

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
        "graph_replay": None if graph_ms_per_step is None else {
            "us_per_step": graph_ms_per_step * 1e3,
            "value": whole_job_levels_per_second(world, B, D, graph_ms_per_step), "unit": UNIT,
            "note": "the step's 21 launches captured once in a CUDA graph and replayed"},
        "lazy_accept": {"us_per_step": lazy_ms_per_step * 1e3,
                        "value": whole_job_levels_per_second(world, B, D, lazy_ms_per_step), "unit": UNIT,
                        "note": "c2t_accept_lazy: accept_len+1 target rows per sequence instead of all final nodes"},
        "single_sequence": single_seq,
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
                     "fp32_logits_full_level": None if fp32_level is None else dict(
                         fp32_level, frac=fp32_level["gbs"] / peak)},
        "cpu_baseline": {"value": cpu_value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def expand_full_level_fp32(c2t, dev, weights, root, prefix, stream, reps: int = 20):
    """Times expand_pass_kernel<fp32> on full levels of the workload with fp32 logits (levels 1-3, three distinct
    buffers of 328 MB, so every launch reads from DRAM).  Returns None if the frontier does not fill."""
    w = WORKLOAD
    B, V, K, F, N = w["B"], w["V"], w["K"], w["F"], w["N"]
    levels = 4
    w1, b1, w2, b2 = weights
    cfg = c2t.Config(batch=B, vocab=V, dtype=c2t.F32, max_depth=levels, topk=K, frontier_cap=F, budget=N,
                     threshold=w["beta"], hidden=w["hidden"], w1=w1, b1=b1, w2=w2, b2=b2, device=dev.index)
    ctx = c2t.Context(cfg)
    draft = [c2t_inputs.draft_logits(B, F, V, 0, l, torch.float32, device=dev) for l in range(levels)]
    rows = []
    ms = []
    for rep in range(reps + 3):
        ctx.c2t_begin_step(root, prefix, stream)
        for l in range(levels):
            if rep == 0:
                rows.append(int(ctx.c2t_get_view()["frontier_n"].sum().item()))
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            ctx.c2t_expand_level(l, draft[l], stream)
            b.record()
            ctx.c2t_prune(l, stream)
            if rep >= 3 and l >= 1:
                ms.append((a, b))
    torch.cuda.synchronize()
    if min(rows[1:]) != B * F:
        return None
    us = sum(a.elapsed_time(b) for a, b in ms) / len(ms) * 1e3
    nbytes = B * F * V * 4
    return {"rows": B * F, "bytes": nbytes, "us": us, "gbs": nbytes / (us * 1e-6) / 1e9}


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


def run_profile(args) -> None:
    """Levels 0 and 1 of the workload (64 + 640 logits rows) and the tail of the step, `steps` times."""
    import paper_2502_13652_b200 as c2t
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = WORKLOAD
    B, V, D, K, F, N = w["B"], w["V"], w["D"], w["K"], w["F"], w["N"]
    w1, b1, w2, b2 = make_weights(w["hidden"])
    cfg = c2t.Config(batch=B, vocab=V, dtype=c2t.BF16, max_depth=D, topk=K, frontier_cap=F, budget=N,
                     threshold=w["beta"], hidden=w["hidden"], w1=w1, b1=b1, w2=w2, b2=b2)
    ctx = c2t.Context(cfg)
    draft = [c2t_inputs.draft_logits(B, F, V, 0, l, torch.bfloat16, device=dev) for l in range(2)]
    target = c2t_inputs.target_logits(B, ctx.Nw, V, 0, torch.bfloat16, device=dev)
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
