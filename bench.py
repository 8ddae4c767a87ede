#!/usr/bin/env python
"""Benchmark of the STTM token-merging path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload long]

One step = one pass of the whole path (spatial quadtree search, temporal linking, root
resolution, ordering, averaging into a packed output) over one synthetic video of the
named workload, through the C ABI (sttm_merge_ex).  The default workload is the
1024-frame, 13x13, D=3584 bf16 video (1.24 GB, ten times the L2) with the thresholds
stored for it.  With N > 1 every rank merges its own copy of the video (independent
videos, no data-path collective); the time is the maximum over ranks.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2507_07990_b200 import inputs  # noqa: E402

METRIC = "input visual tokens/sec merged on 1 B200; achieved HBM GB/s vs peak"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of a kernel as a multiple of its algorithmic bytes, from the ncu capture
# summarised under profiles/ (dram__bytes_read.sum + dram__bytes_write.sum on the qwen workload;
# a streaming kernel's traffic grows in proportion to the bytes it must move, so the ratio is
# applied to the benchmark workload's algorithmic bytes).  Absent = no capture of the current kernel.
NCU_TRAFFIC_RATIO = {"fused": 0.946}


def workload_setup(name: str):
    cfg = inputs.CONFIGS[name]
    table = inputs.load_thresholds()[name]
    spec = inputs.config_videos(name, table.get("seed_bump", 0))[0]
    per_budget = table["videos"][0]
    key = "fixed" if "fixed" in per_budget else "%.2f" % cfg["budgets"][-1]
    th = per_budget[key]
    return cfg, spec, th, key


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """SM clock and throttle reasons while the timed region runs, read through NVML every few
    milliseconds from a thread (reading only: nothing on the GPU is set)."""
    REASONS = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40, "sw_power_cap": 0x4}

    def __init__(self, index: int, period_s: float = 0.004):
        import threading
        self.samples, self.max_mhz, self.bits = [], None, 0
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = int(visible.split(",")[index]) if visible and visible.split(",")[index].isdigit() else index
            self._h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None
            return

        def loop():
            while not self._stop.is_set():
                try:
                    self.samples.append(float(self._nv.nvmlDeviceGetClockInfo(self._h, self._nv.NVML_CLOCK_SM)))
                    self.bits |= int(self._nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                except Exception:
                    pass
                self._stop.wait(period_s)

        self._thread = threading.Thread(target=loop, daemon=True)
        self._thread.start()

    def stop(self):
        if self._nv is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["NVML unavailable"]}
        self._stop.set()
        self._thread.join(timeout=2)
        reasons = sorted(n for n, b in self.REASONS.items() if self.bits & b)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "samples": len(self.samples), "reasons": reasons}


def cpu_baseline(video_np, th, frames):
    """The oracle as it stands, on the host cores, on the first `frames` frames."""
    from oracle import oracle
    sample = video_np[:frames]
    t0 = time.perf_counter()
    r = oracle.merge(sample, th["tau_s"], th["tau_t"], want_feats=True)
    dt = time.perf_counter() - t0
    tokens = sample.shape[0] * sample.shape[1] * sample.shape[2]
    # want_feats runs the structure pass twice (once to size the output buffer)
    return {"value": tokens / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": "first %d of %d frames (%d tokens), one thread, fp64, %.2f s, %d rows"
                      % (sample.shape[0], video_np.shape[0], tokens, dt, r.count)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    cfg, spec, th, key = workload_setup(args.workload)
    frames = min(spec.T, args.reference_frames)
    import dataclasses
    video = inputs.make_video(dataclasses.replace(spec, T=frames))
    from oracle import oracle
    tokens = frames * spec.H * spec.W
    for _ in range(args.warmup):
        oracle.merge(video, th["tau_s"], th["tau_t"], want_feats=True)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.merge(video, th["tau_s"], th["tau_t"], want_feats=True)
    dt = time.perf_counter() - t0
    value = tokens * args.steps / dt
    sample = "first %d of %d frames (%d tokens) per step, one thread, fp64" % (frames, spec.T, tokens)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(args.workload, spec, th, key),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def workload_config(name, spec, th, key):
    return {"workload": "%s: 1 video/GPU, T=%d, %dx%d grid, D=%d %s, block generator p_static=%.2f sigma=%.2f"
                        % (name, spec.T, spec.H, spec.W, spec.D, spec.dtype, spec.p_static, spec.sigma),
            "budget": key, "tau_s": th["tau_s"], "tau_t": th["tau_t"], "lv1": 4,
            "kept_fraction": th["fraction"], "out_rows": th["count"],
            "l2": "input (%.0f MB) larger than L2; no flush" % (spec.tokens * spec.D * 2 / 1e6)
                  if spec.tokens * spec.D * 2 > 200e6 else "L2 flushed between steps"}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2507_07990_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    tuning = [int(v) for v in args.tuning.split(",")]
    binding.load_library().sttm_set_tuning(*tuning[:3])
    if len(tuning) > 3:
        binding.load_library().sttm_set_ring_split(*(tuning[3:5] + [0])[:2])

    cfg, spec, th, key = workload_setup(args.workload)
    N = spec.tokens
    in_bytes = N * spec.D * (2 if spec.dtype == "bf16" else 4)
    small = in_bytes <= 200e6
    tdtype = torch.bfloat16 if spec.dtype == "bf16" else torch.float32

    # the video, generated once into pinned host memory and copied to the device
    h_feats = torch.empty((1, spec.T, spec.H, spec.W, spec.D), dtype=tdtype).pin_memory()
    view = h_feats.view(torch.int16).numpy().view(np.uint16) if spec.dtype == "bf16" else h_feats.numpy()
    inputs.make_video(spec, out=view[0])
    d_feats = h_feats.cuda()
    if args.budget_rows > 0:
        # budget mode: tau_t chosen on the device for this many rows (two passes of the fused kernel)
        plan = binding.BudgetPlan((1, spec.T, spec.H, spec.W, spec.D), tdtype, th["tau_s"], args.budget_rows,
                                  out_dtype=torch.bfloat16, want_map=False)
    else:
        plan = binding.MergePlan((1, spec.T, spec.H, spec.W, spec.D), tdtype, th["tau_s"], th["tau_t"],
                                 out_dtype=torch.bfloat16, want_map=False,
                                 match=binding.MATCH_BEST if args.match == "best" else binding.MATCH_TOPLEFT)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if small else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    out = None
    for _ in range(max(args.warmup, 3)):
        out = plan.run(d_feats)
    torch.cuda.synchronize()
    count = int(out.out_count[0].item())
    status = int(out.device_status.item())
    if status != 0:
        raise RuntimeError("device status %d" % status)
    launches_per_step = out.launches

    # The step is also captured once as a CUDA graph (the same kernels, launched by one replay
    # instead of nine calls).  Every fourth timed step goes through the library call with stage
    # events set (they give the kernels' own durations), the others replay the graph.
    graph = None
    if not args.no_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                plan.run(d_feats)
            torch.cuda.current_stream().wait_stream(side)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                plan.run(d_feats)
            graph.replay()
            torch.cuda.synchronize()
            if int(plan.out_count[0].item()) != count or int(plan.status.item()) != 0:
                raise RuntimeError("graph replay gave another result")
        except Exception as exc:          # capture not possible here: every step is a direct call
            print("bench: no CUDA graph (%s)" % exc, file=sys.stderr)
            graph = None
    sampled = [k for k in range(args.steps) if graph is None or k % 4 == 0]
    timers = {k: binding.StageTimer() for k in sampled}
    lib = binding.load_library()
    step_events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(args.steps)]
    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    for k in range(args.steps):
        if flush is not None:
            flush.fill_(k & 0xff)
        if k in timers:
            lib.sttm_set_stage_events(timers[k]._handles)
            step_events[k][0].record()
            plan.run(d_feats)
            step_events[k][1].record()
            lib.sttm_set_stage_events(None)
        else:
            step_events[k][0].record()
            graph.replay()
            step_events[k][1].record()
    barrier()
    clocks = sampler.stop() if sampler is not None else None
    step_ms = [a.elapsed_time(b) for a, b in step_events]
    total_ms = torch.tensor([sum(step_ms)], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(total_ms, op=dist.ReduceOp.MAX)
    total_ms = float(total_ms.item())
    ms_per_step = total_ms / args.steps
    value = world * N * args.steps / (total_ms / 1e3)

    # per-stage times over the sampled steps of the timed region (events on the launching stream)
    stage_ms = {}
    for tm in timers.values():
        for n, v in tm.stage_ms().items():
            stage_ms[n] = stage_ms.get(n, 0.0) + v / len(timers)
    out_bytes = count * spec.D * 2
    id_bytes = count * 4
    path_bytes = in_bytes + out_bytes + id_bytes
    # algorithmic bytes per launch of each feature-touching stage: every stage of the three-pass
    # kernels reads the input once; the fused kernel reads it once and writes every output row once
    # (to its staging place), the gather moves every output row once more
    if lib.sttm_last_path() == 3:
        stage_bytes = {"gram": in_bytes, "sum": in_bytes + out_bytes}
    elif lib.sttm_last_path() == 1:
        stage_bytes = {"fused": in_bytes + out_bytes, "gather": 2 * out_bytes}
    else:
        stage_bytes = {"spatial": in_bytes, "temporal+roots": in_bytes, "accumulate": in_bytes + out_bytes}
    dominant = max(stage_bytes, key=lambda n: stage_ms.get(n, 0.0))
    peak, peak_kind = measured_peak()
    achieved = stage_bytes[dominant] / (stage_ms[dominant] / 1e3) / 1e9
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": "of " + peak_kind,
                "traffic": (NCU_TRAFFIC_RATIO[dominant] * stage_bytes[dominant]
                            if dominant in NCU_TRAFFIC_RATIO else None),
                "algorithmic_bytes": stage_bytes[dominant], "kernel_ms": stage_ms[dominant],
                "stage_ms": stage_ms,
                "path": {"algorithmic_bytes": path_bytes, "achieved": path_bytes / (ms_per_step / 1e3) / 1e9,
                         "frac": path_bytes / (ms_per_step / 1e3) / 1e9 / peak,
                         "frac_of_8000": path_bytes / (ms_per_step / 1e3) / 1e9 / 8000.0}}

    # end to end through the host-buffer entry point: H2D of the video, D2H of the result
    e2e_steps = max(1, min(args.steps, 5 if not small else args.steps))
    h_out = torch.empty((N, spec.D), dtype=torch.bfloat16).pin_memory()
    h_pos = torch.empty((N,), dtype=torch.int32).pin_memory()
    binding.sttm_merge_host(h_feats, th["tau_s"], th["tau_t"], h_out_feats=h_out, h_out_pos=h_pos)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        r = binding.sttm_merge_host(h_feats, th["tau_s"], th["tau_t"], h_out_feats=h_out, h_out_pos=h_pos)
    barrier()
    e2e_s = torch.tensor([time.perf_counter() - t0], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(e2e_s, op=dist.ReduceOp.MAX)
    e2e = {"value": world * N * e2e_steps / float(e2e_s.item()), "unit": UNIT, "h2d_bytes_per_step": in_bytes,
           "d2h_bytes_per_step": out_bytes + id_bytes + 4 + 16, "steps": e2e_steps,
           "ms_per_step": 1e3 * float(e2e_s.item()) / e2e_steps}
    assert int(r.out_count[0]) == count

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": dict(workload_config(args.workload, spec, th, key),
                               match=args.match, budget_rows=args.budget_rows,
                               launch=("3 of 4 steps replay a CUDA graph of the library call, every 4th is the call "
                                       "itself with stage events") if graph is not None else "library calls"),
                "out_rows": count,
                "launch_shape": binding.sttm_fused_launch_shape(plan.problem),
                "roofline": roofline, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
                "clocks": clocks}
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(view[0], th, min(spec.T, args.baseline_frames))
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long", choices=list(inputs.CONFIGS))
    ap.add_argument("--baseline-frames", type=int, default=512,
                    help="frames of the workload the CPU-baseline leg runs the oracle on")
    ap.add_argument("--reference-frames", type=int, default=64,
                    help="frames per step of the --impl reference arm")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="every timed step is a direct library call")
    ap.add_argument("--budget-rows", type=int, default=0,
                    help="time the budget mode (sttm_merge_budget) with this row budget instead of fixed thresholds")
    ap.add_argument("--match", default="topleft", choices=["topleft", "best"],
                    help="destination rule of the temporal link (the paper's default, or its most-similar variant)")
    ap.add_argument("--tuning", default="0,0,0",
                    help="path,cluster_size,frames_per_item for sttm_set_tuning, optionally followed by "
                         "sum_slots,lead_frames for sttm_set_ring_split (0 = library's choice)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
