#!/usr/bin/env python
"""Benchmark of the STTM token-merging path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload long|llava|qwen|mixed|tiny] [--budget 0.3|0.5]

One step = one pass of the whole path (spatial quadtree search, temporal linking, root
resolution, ordering, averaging into a packed output) over the synthetic videos of the named
workload, through the C ABI (one sttm_merge_ex call; the `mixed` workload is one call on its
batch of eight videos with per-video thresholds).  The default workload is the 1024-frame,
13x13, D=3584 bf16 video (1.24 GB, ten times the L2) at the thresholds stored for its 30 %
token budget.  With N > 1 every rank merges its own copy of the workload (independent
videos, no data-path collective); the time is the maximum over ranks.  Without a launcher
(`WORLD_SIZE` unset) `--gpus N` starts the N ranks itself.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import statistics
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
PROFILE_DIR = os.path.join(ROOT, "profiles")


def ncu_traffic_ratio(kernel: str):
    """DRAM traffic of a kernel as a multiple of its algorithmic bytes, as an ncu summary under
    profiles/ states it (a line `dram_traffic_ratio <kernel> = <number>`); None when no summary
    has such a line, i.e. there is no capture of the kernel as it stands."""
    try:
        for name in sorted(os.listdir(PROFILE_DIR)):
            if not name.endswith((".md", ".txt")):
                continue
            with open(os.path.join(PROFILE_DIR, name)) as f:
                m = re.search(r"dram_traffic_ratio\s+%s\s*=\s*([0-9.]+)" % re.escape(kernel), f.read())
            if m:
                return float(m.group(1))
    except OSError:
        pass
    return None


def workload_setup(name: str, budget=None):
    """(config, specs, thresholds per video, budget key) of a named workload."""
    cfg = inputs.CONFIGS[name]
    table = inputs.load_thresholds()[name]
    specs = inputs.config_videos(name, table.get("seed_bump", 0))
    if "fixed" in table["videos"][0]:
        key = "fixed"
    else:
        key = "%.2f" % (budget if budget is not None else cfg["budgets"][-1])
        if key not in table["videos"][0]:
            raise SystemExit("workload %s has no thresholds for budget %s (has %s)" % (name, key, sorted(table["videos"][0])))
    ths = [v[key] for v in table["videos"]]
    return cfg, specs, ths, key


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """SM clock and throttle reasons while the timed region runs, read through NVML every
    millisecond or two from a thread (reading only: nothing on the GPU is set)."""
    REASONS = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40, "sw_power_cap": 0x4}

    def __init__(self, index: int, period_s: float = 0.001):
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


def oracle_on_cores(video_np, th, chunk_frames, max_threads=None):
    """The oracle as it stands on the host cores this process may use: the sample is cut into
    runs of `chunk_frames` frames and every thread runs the whole oracle on its own run (the C
    code releases the interpreter lock).  Chains that would cross a cut are cut, which changes
    the row count a little and the work not at all.  Returns (tokens/s, threads, seconds, rows, frames)."""
    import concurrent.futures as cf
    from oracle import oracle
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    threads = max(1, min(cores, video_np.shape[0] // chunk_frames, max_threads or cores))
    chunks = [video_np[i * chunk_frames:(i + 1) * chunk_frames] for i in range(threads)]
    oracle.merge(chunks[0][:2], th["tau_s"], th["tau_t"], want_feats=True)          # load the library first

    def work(c):
        return oracle.merge(c, th["tau_s"], th["tau_t"], want_feats=True).count

    t0 = time.perf_counter()
    with cf.ThreadPoolExecutor(max_workers=threads) as ex:
        rows = sum(ex.map(work, chunks))
    dt = time.perf_counter() - t0
    frames = threads * chunk_frames
    tokens = frames * video_np.shape[1] * video_np.shape[2]
    return tokens / dt, threads, dt, rows, frames


def cpu_baseline(video_np, th, chunk_frames):
    value, threads, dt, rows, frames = oracle_on_cores(video_np, th, chunk_frames)
    one, _, dt1, _, _ = oracle_on_cores(video_np, th, chunk_frames, max_threads=1)
    return {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
            "cores_available": len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count(),
            "one_thread": one,
            "sample": "first %d of %d frames of video 0, %d threads x %d frames each, fp64, %.2f s (one thread on "
                      "%d frames: %.2f s), %d rows" % (frames, video_np.shape[0], threads, chunk_frames, dt,
                                                       chunk_frames, dt1, rows)}


def workload_config(name, specs, ths, key):
    spec = specs[0]
    in_bytes = sum(s.tokens * s.D * (2 if s.dtype == "bf16" else 4) for s in specs)
    tokens = sum(s.tokens for s in specs)
    rows = sum(t["count"] for t in ths)
    return {"workload": "%s: %d video%s/GPU, T=%d, %dx%d grid, D=%d %s, block generator p_static=%s sigma=%.2f, "
                        "contrast classes %s"
                        % (name, len(specs), "" if len(specs) == 1 else "s in one call", spec.T, spec.H, spec.W, spec.D,
                           spec.dtype, "/".join("%.2f" % s.p_static for s in specs), spec.sigma, list(spec.contrast)),
            "budget": key, "tau_s": [t["tau_s"] for t in ths], "tau_t": [t["tau_t"] for t in ths], "lv1": 4,
            "kept_fraction": rows / tokens, "out_rows": rows, "rows_per_video": [t["count"] for t in ths],
            "l2": "input (%.0f MB) larger than L2; no flush" % (in_bytes / 1e6) if in_bytes > 200e6
                  else "L2 flushed between steps"}


def run_reference(args):
    """The reference arm: there is no reference implementation (the reference is a paper), so this
    times the CPU oracle, as it stands, on a bounded sample of the workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    cfg, specs, ths, key = workload_setup(args.workload, args.budget)
    spec, th = specs[0], ths[0]
    frames = min(spec.T, args.reference_frames)
    import dataclasses
    video = inputs.make_video(dataclasses.replace(spec, T=frames))
    chunk = max(2, min(frames, 32))
    for _ in range(args.warmup):
        oracle_on_cores(video, th, chunk)
    t0 = time.perf_counter()
    used = 0
    for _ in range(args.steps):
        _, threads, _, _, used = oracle_on_cores(video, th, chunk)
    dt = time.perf_counter() - t0
    tokens = used * spec.H * spec.W
    value = tokens * args.steps / dt
    sample = "first %d of %d frames of video 0 (%d tokens) per step, %d threads x %d frames, fp64" % (
        used, spec.T, tokens, threads, chunk)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(args.workload, specs, ths, key),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def spawn_selftest(rank, world, port):
    """CPU check of the rank start-up: gloo ranks, a max over ranks, one line from rank 0."""
    import torch
    import torch.distributed as dist
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    t = torch.tensor([float(rank + 1)], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "selftest": True, "n_gpus": world, "max_over_ranks": float(t.item())}))
    dist.destroy_process_group()


def _spawned(rank, world, port, argv):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    sys.argv = argv
    args = parse_args()
    if args.selftest_spawn:
        return spawn_selftest(rank, world, port)
    (run_segments if args.mode == "segments" else run_ours)(args)


def spawn_ranks(args):
    """`--gpus N` without a launcher: start the N ranks here (one process per GPU, NCCL)."""
    import socket
    import torch
    import torch.multiprocessing as mp
    if not args.selftest_spawn and torch.cuda.device_count() < args.gpus:
        raise SystemExit("bench.py --gpus %d: only %d CUDA devices visible" % (args.gpus, torch.cuda.device_count()))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_spawned, args=(args.gpus, port, list(sys.argv)), nprocs=args.gpus, join=True)
    return 0


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
    lib = binding.load_library()
    tuning = [int(v) for v in args.tuning.split(",")]
    lib.sttm_set_tuning(*tuning[:3])
    if len(tuning) > 3:
        lib.sttm_set_ring_split(*(tuning[3:5] + [0])[:2])

    cfg, specs, ths, key = workload_setup(args.workload, args.budget)
    spec = specs[0]
    B = len(specs)
    N = sum(s.tokens for s in specs)
    elt = 2 if spec.dtype == "bf16" else 4
    in_bytes = N * spec.D * elt
    small = in_bytes <= 200e6
    tdtype = torch.bfloat16 if spec.dtype == "bf16" else torch.float32
    tau_s = [t["tau_s"] for t in ths] if B > 1 else ths[0]["tau_s"]
    tau_t = [t["tau_t"] for t in ths] if B > 1 else ths[0]["tau_t"]

    # the videos, generated once into pinned host memory and copied to the device
    shape = (B, spec.T, spec.H, spec.W, spec.D)
    h_feats = torch.empty(shape, dtype=tdtype).pin_memory()
    view = h_feats.view(torch.int16).numpy().view(np.uint16) if spec.dtype == "bf16" else h_feats.numpy()
    for b, s in enumerate(specs):
        inputs.make_video(s, out=view[b])
    d_feats = h_feats.cuda()
    if args.budget_rows > 0:
        # budget mode: tau_t chosen on the device for this many rows per video
        plan = binding.BudgetPlan(shape, tdtype, tau_s, args.budget_rows, out_dtype=torch.bfloat16, want_map=False)
    else:
        plan = binding.MergePlan(shape, tdtype, tau_s, tau_t, out_dtype=torch.bfloat16, want_map=False,
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
    counts = [int(v) for v in out.out_count.tolist()]
    count = sum(counts)
    status = int(out.device_status.item())
    if status != 0:
        raise RuntimeError("device status %d" % status)
    if args.budget_rows == 0 and args.match == "topleft" and counts != [t["count"] for t in ths]:
        raise RuntimeError("row counts %s differ from the calibrated %s" % (counts, [t["count"] for t in ths]))
    launches_per_step = out.launches

    # The step is also captured once as a CUDA graph (the same kernels, launched by one replay
    # instead of one call per kernel).  Every fourth timed step goes through the library call, every
    # eighth with stage events set (they give the kernels' own durations), the others replay the graph.
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
            if int(plan.out_count.sum().item()) != count or int(plan.status.item()) != 0:
                raise RuntimeError("graph replay gave another result")
        except Exception as exc:          # capture not possible here: every step is a direct call
            print("bench: no CUDA graph (%s)" % exc, file=sys.stderr)
            graph = None
    # (stage events between two kernels keep the later one from becoming resident under the earlier one,
    # so only every second direct call carries them; the others are what a caller of the library sees)
    sampled = [k for k in range(args.steps) if graph is None or k % 4 == 0]
    staged = sampled[::2]
    timers = {k: binding.StageTimer() for k in staged}
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
        elif k in sampled:
            step_events[k][0].record()
            plan.run(d_feats)
            step_events[k][1].record()
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
    direct_ms = [step_ms[k] for k in sampled if k not in timers] or [step_ms[k] for k in sampled]
    replay_ms = [step_ms[k] for k in range(args.steps) if k not in sampled]

    # per-stage times over the sampled steps of the timed region (events on the launching stream)
    stage_ms = {}
    for tm in timers.values():
        for n, v in tm.stage_ms().items():
            stage_ms[n] = stage_ms.get(n, 0.0) + v / len(timers)
    out_bytes = count * spec.D * 2
    id_bytes = count * 4
    path_bytes = in_bytes + out_bytes + id_bytes
    # algorithmic bytes per launch of each feature-touching stage: the single-pass kernel reads the
    # input once and writes every output row once (to its staging place), its gather moves every row
    # once more; the Gram stage of the two-stream kernels reads the input, their sum stage reads it
    # again and writes every row; every stage of the three-pass kernels reads the input once
    path_id = lib.sttm_last_path()
    if path_id == 3:
        stage_bytes = {"gram": in_bytes, "sum": in_bytes + out_bytes}
    elif path_id == 1:
        stage_bytes = {"fused": in_bytes + out_bytes, "gather": 2 * out_bytes}
    else:
        stage_bytes = {"spatial": in_bytes, "temporal+roots": in_bytes, "accumulate": in_bytes + out_bytes}
    dominant = max(stage_bytes, key=lambda n: stage_ms.get(n, 0.0))
    peak, peak_kind = measured_peak()
    achieved = stage_bytes[dominant] / (stage_ms[dominant] / 1e3) / 1e9
    ratio = ncu_traffic_ratio(dominant)
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": "of " + peak_kind,
                "traffic": ratio * stage_bytes[dominant] if ratio is not None else None,
                "algorithmic_bytes": stage_bytes[dominant], "kernel_ms": stage_ms[dominant],
                "stage_ms": stage_ms,
                "path": {"algorithmic_bytes": path_bytes, "achieved": path_bytes / (ms_per_step / 1e3) / 1e9,
                         "frac": path_bytes / (ms_per_step / 1e3) / 1e9 / peak,
                         "frac_of_8000": path_bytes / (ms_per_step / 1e3) / 1e9 / 8000.0}}

    # end to end through the host-buffer entry point: H2D of the videos, D2H of the result
    e2e_steps = max(1, min(args.steps, 5 if not small else args.steps))
    h_out = torch.empty((N, spec.D), dtype=torch.bfloat16).pin_memory()
    h_pos = torch.empty((N,), dtype=torch.int32).pin_memory()
    e2e_tau_t = tau_t
    if args.budget_rows > 0:
        e2e_tau_t = [float(v) for v in plan.tau.tolist()] if B > 1 else float(plan.tau[0].item())
    binding.sttm_merge_host(h_feats, tau_s, e2e_tau_t, h_out_feats=h_out, h_out_pos=h_pos)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        r = binding.sttm_merge_host(h_feats, tau_s, e2e_tau_t, h_out_feats=h_out, h_out_pos=h_pos)
    barrier()
    e2e_s = torch.tensor([time.perf_counter() - t0], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(e2e_s, op=dist.ReduceOp.MAX)
    e2e = {"value": world * N * e2e_steps / float(e2e_s.item()), "unit": UNIT, "h2d_bytes_per_step": in_bytes,
           "d2h_bytes_per_step": out_bytes + id_bytes + 4 * B + 8 * (B + 1) + 4, "steps": e2e_steps,
           "ms_per_step": 1e3 * float(e2e_s.item()) / e2e_steps}
    assert int(sum(r.out_count)) == count

    if rank == 0:
        mhz = clocks["sm_mhz"] if clocks else None
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
                "ms_median": statistics.median(step_ms), "ms_best": min(step_ms),
                "ms_direct_call": statistics.mean(direct_ms) if direct_ms else None,
                "ms_graph_replay": statistics.mean(replay_ms) if replay_ms else None,
                "ms_x_mhz": ms_per_step * mhz if mhz else None,
                "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": dict(workload_config(args.workload, specs, ths, key),
                               match=args.match, budget_rows=args.budget_rows,
                               launch=("3 of 4 steps replay a CUDA graph of the library call, every 4th is the call "
                                       "itself, every 8th with stage events") if graph is not None
                               else "library calls, every 2nd with stage events"),
                "out_rows": count, "rows_per_video": counts,
                "launch_shape": binding.sttm_fused_launch_shape(plan.problem),
                "roofline": roofline, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
                "clocks": clocks}
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(view[0], ths[0], min(spec.T, args.baseline_frames))
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_segments(args):
    """`--mode segments`: ONE video cut into runs of consecutive frames, one run per rank
    (segments.SegmentMerge + DistLink: every rank merges its frames with the last frame of the rank
    before in front, then one message per cut travels from the last rank to the first).  The ranks'
    rows and ids, put together, are checked against the merge of the whole video on rank 0's GPU."""
    import torch
    import torch.distributed as dist
    from paper_2507_07990_b200 import binding, segments

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if "MASTER_ADDR" in os.environ:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        import socket
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % port, rank=0, world_size=1,
                                device_id=torch.device("cuda", local))
    lib = binding.load_library()
    cfg, specs, ths, key = workload_setup(args.workload, args.budget)
    if len(specs) != 1:
        raise SystemExit("--mode segments cuts one video; workload %s holds %d" % (args.workload, len(specs)))
    spec, th = specs[0], ths[0]
    if spec.dtype != "bf16":
        raise SystemExit("--mode segments runs the bf16 workloads")
    HW = spec.H * spec.W
    video = inputs.make_video(spec)                     # every rank generates the video and keeps its own frames
    cuts = segments.cut_frames(spec.T, world)
    a, b = cuts[rank], cuts[rank + 1]
    halo = 1 if rank > 0 else 0
    mine = torch.from_numpy(video[a - halo:b].view(np.int16)).view(torch.bfloat16).cuda()
    part = segments.SegmentMerge(mine, bool(halo), a, th["tau_s"], th["tau_t"], out_dtype=torch.bfloat16)
    link = segments.DistLink()

    def barrier():
        dist.barrier()
        torch.cuda.synchronize()

    out = None
    for _ in range(max(args.warmup, 3)):
        part.merge_local()
        out = part.finish(link)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    ev0.record()
    for _ in range(args.steps):
        part.merge_local()
        out = part.finish(link)
    ev1.record()
    barrier()
    clocks = sampler.stop() if sampler is not None else None
    # kernels per step: the merge of the segment, of its halo frame, and the fold / emit / finish kernels
    launches = args.steps * (part.res.launches + (part.halo.launches + 1 if halo else 0) + (1 if rank + 1 < world else 0) + 1)
    total_ms = torch.tensor([ev0.elapsed_time(ev1)], dtype=torch.float64, device="cuda")
    dist.all_reduce(total_ms, op=dist.ReduceOp.MAX)
    total_ms = float(total_ms.item())
    if int(out.device_status.item()) != 0:
        raise RuntimeError("device status %d on rank %d" % (int(out.device_status.item()), rank))

    # the packed result: counts and ids of every rank, in rank order
    owned = torch.tensor([out.owned_count], dtype=torch.int64, device="cuda")
    every = [torch.zeros_like(owned) for _ in range(world)]
    dist.all_gather(every, owned)
    counts = [int(c.item()) for c in every]
    ids = torch.full((max(counts + [1]),), -1, dtype=torch.int32, device="cuda")
    ids[:out.owned_count] = out.out_pos[:out.owned_count]
    all_ids = [torch.empty_like(ids) for _ in range(world)]
    dist.all_gather(all_ids, ids)
    check = None
    if rank == 0:
        whole = torch.from_numpy(video.view(np.int16)).view(torch.bfloat16).cuda().unsqueeze(0)
        plan = binding.MergePlan(tuple(whole.shape), torch.bfloat16, th["tau_s"], th["tau_t"], out_dtype=torch.bfloat16,
                                 want_map=False)
        ref = plan.run(whole)
        n = int(ref.out_count[0].item())
        got = torch.cat([t[:c] for t, c in zip(all_ids, counts)])
        check = {"rows": sum(counts), "rows_single_gpu": n, "rows_calibrated": th["count"],
                 "ids_equal": bool(got.numel() == n and torch.equal(got, ref.out_pos[:n]))}
        if not (check["ids_equal"] and n == th["count"]):
            raise RuntimeError("segments disagree with the whole video: %s" % check)
        in_bytes = spec.tokens * spec.D * 2
        line = {"metric": METRIC, "value": spec.tokens * args.steps / (total_ms / 1e3), "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps,
                "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": dict(workload_config(args.workload, specs, ths, key), mode="segments",
                               frames_per_rank=[cuts[r + 1] - cuts[r] for r in range(world)],
                               message="per cut at most %d rows of %d fp32 sums, weights and ids, last rank first"
                                       % (HW, spec.D)),
                "out_rows": sum(counts), "rows_per_rank": counts, "check": check,
                "roofline": None, "e2e": None, "gpu_launches": launches, "clocks": clocks,
                "path": {"algorithmic_bytes": in_bytes + sum(counts) * (spec.D * 2 + 4),
                         "achieved": (in_bytes + sum(counts) * (spec.D * 2 + 4)) / (total_ms / args.steps / 1e3) / 1e9}}
        print(json.dumps(line))
    dist.destroy_process_group()
    return 0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long", choices=list(inputs.CONFIGS))
    ap.add_argument("--budget", type=float, default=None,
                    help="token budget whose stored thresholds are used (0.5 or 0.3; default: the workload's last)")
    ap.add_argument("--baseline-frames", type=int, default=64,
                    help="frames every thread of the CPU-baseline leg runs the oracle on")
    ap.add_argument("--reference-frames", type=int, default=256,
                    help="frames of video 0 the --impl reference arm shares out over its threads per step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="every timed step is a direct library call")
    ap.add_argument("--budget-rows", type=int, default=0,
                    help="time the budget mode (sttm_merge_budget) with this row budget per video instead of fixed thresholds")
    ap.add_argument("--match", default="topleft", choices=["topleft", "best"],
                    help="destination rule of the temporal link (the paper's default, or its most-similar variant)")
    ap.add_argument("--tuning", default="0,0,0",
                    help="path,cluster_size,frames_per_item for sttm_set_tuning (path 5: the two-stream kernels, 6: the same with the mma.sync Gram stage, 2: the single-pass kernel), "
                         "optionally followed by sum_slots,lead_frames for sttm_set_ring_split (0 = library's choice)")
    ap.add_argument("--mode", default="videos", choices=["videos", "segments"],
                    help="videos: every rank merges its own videos (the default); segments: one video cut by frames "
                         "over the ranks, checked against the merge of the whole video")
    ap.add_argument("--selftest-spawn", action="store_true", help=argparse.SUPPRESS)
    return ap.parse_args()


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if "WORLD_SIZE" not in os.environ and (args.gpus > 1 or args.selftest_spawn):
        return spawn_ranks(args)
    return (run_segments if args.mode == "segments" else run_ours)(args)


if __name__ == "__main__":
    sys.exit(main())
