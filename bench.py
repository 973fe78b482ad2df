#!/usr/bin/env python
"""Throughput of the TTF pass on B200: visual tokens/s and clips/s through ttf_compress, roofline fraction of
the dominant kernel, end-to-end rate through the host-buffer entry point, and the CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload NAME] [--clips B] [--streams S] [--no-e2e] [--no-cpu]

A step is one pass of the whole path (norm/frame-sum sweep, anchor pick, windowed match + gate, compaction
with positions and fuse bookkeeping) over a batch of B distinct synthetic clips of the workload: one
ttf_compress_batch call (or, with --streams S, one ttf_compress call per clip on S streams of the caller).
The batch is larger than L2, so every clip starts cold in HBM.  Rank 0 prints
one JSON line.  With N > 1 (torchrun) every rank runs the same batch shape on its own GPU: clips are
independent, there is no collective on the data path (weak scaling, replicas).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "visual tokens/s through TTF"
UNIT = "tokens/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vl8b_cal")
    ap.add_argument("--clips", type=int, default=16, help="distinct clips per step (batch)")
    ap.add_argument("--streams", type=int, default=0,
                    help="0: one ttf_compress_batch call per step (the library spreads the clips over its own "
                         "streams, see --lanes); S > 0: one ttf_compress call per clip on S streams of the caller")
    ap.add_argument("--lanes", type=int, default=0, help="clips of a batch in flight (ttf_set_schedule); 0 = automatic, -1 = the pipelined schedule")
    ap.add_argument("--match-kernel", default="auto", choices=["auto", "mma", "tc"],
                    help="kernel of the matching step for bf16 clips (ttf_set_match_kernel)")
    ap.add_argument("--threshold", type=float, default=None)
    ap.add_argument("--anchor", default="auto", choices=["auto", "first", "last"], help="anchor rule")
    ap.add_argument("--no-graph", action="store_true",
                    help="launch every kernel from the host each step instead of replaying a captured CUDA graph")
    ap.add_argument("--ncu-range", action="store_true",
                    help="profiling aid: after the warm-up run ONE step between cudaProfilerStart/Stop and exit without "
                         "timing anything (for `ncu --replay-mode range`, which measures the overlapped kernels of the "
                         "step as one workload)")
    ap.add_argument("--extensions", action="store_true",
                    help="time the extension entry points (restore, streaming segment, histogram, mean fuse) instead of "
                         "the compression pass and print one JSON line with their roofline fractions")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    return ap.parse_args()


def stored_traffic(workload: str, kernel: str, csrc: str):
    """DRAM bytes (read + write) per launch of `kernel` from the stored profiler counters, or None when there are
    none for this workload or they were taken on other sources than the library was built from."""
    path = os.path.join(ROOT, "profiles", f"dram_per_kernel_{workload}.json")
    try:
        d = json.load(open(path))
    except Exception:
        return None, "no stored counters for this workload"
    if d.get("csrc_hash") != csrc:
        return None, "stored counters were taken on other kernel sources"
    k = d.get("kernels", {}).get(kernel)
    if not k:
        return None, "no stored counters for this kernel"
    return int(k["dram_bytes_read"]) + int(k["dram_bytes_write"]), d.get("note", "ncu, one launch")


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


# ---------------------------------------------------------------------------------------------------------
# clock sampling (reads only; never changes a GPU setting)
# ---------------------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, torch_device: int, period_s: float = 0.004):
        self.samples = []           # (time, sm_mhz, reasons bitmask)
        self.period = period_s
        self.handle = None
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_device).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception as e:      # no NVML: the JSON says so
            self.error = repr(e)

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
                try:
                    rs = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                except Exception:
                    rs = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                self.samples.append((time.perf_counter(), mhz, rs))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.handle is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self, t0: float, t1: float) -> dict:
        if self.handle is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML unavailable"}
        window = "timed"
        sel = [s for s in self.samples if t0 <= s[0] <= t1]
        if len(sel) < 3:
            sel, window = self.samples, "run"
        if not sel:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "note": "no samples"}
        bits = 0
        for _, _, rs in sel:
            bits |= rs
        reasons = sorted(name for bit, name in self.REASONS.items() if bits & bit)
        return {"sm_mhz": statistics.median(s[1] for s in sel), "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(sel), "window": window}


# ---------------------------------------------------------------------------------------------------------
# reference arm / CPU baseline: the oracle as it stands, on the host cores
# ---------------------------------------------------------------------------------------------------------
def oracle_sample_plan(spec, t, budget_s_per_step):
    """Times the oracle on one clip, then sizes a step's sample to the budget."""
    from oracle import ttf_oracle as O
    from paper_2605_07355_b200 import clips
    X = clips.make_clip(spec, spec.seed)
    t0 = time.perf_counter()
    O.compress(X, spec.r, t)
    one = time.perf_counter() - t0
    if one <= budget_s_per_step:
        n = max(1, min(4, int(budget_s_per_step / one)))
        Xs = [X] + [clips.make_clip(spec, spec.seed + j) for j in range(1, n)]
        desc = f"{n} whole clip(s) of {spec.name} per step"
    else:
        frames = max(2, int(spec.F * budget_s_per_step / one))
        Xs = [np.ascontiguousarray(X[:frames])]
        desc = f"first {frames} of {spec.F} frames of one {spec.name} clip per step"
    return Xs, desc


def run_oracle_steps(Xs, spec, t, steps, warmup):
    from oracle import ttf_oracle as O
    tokens = sum(x.shape[0] * x.shape[1] * x.shape[2] for x in Xs)
    for _ in range(warmup):
        for x in Xs:
            O.compress(x, spec.r, t)
    t0 = time.perf_counter()
    for _ in range(steps):
        for x in Xs:
            O.compress(x, spec.r, t)
    dt = time.perf_counter() - t0
    return tokens * steps / dt, dt / steps * 1e3, tokens


def reference_arm(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import ttf_oracle as O
    from paper_2605_07355_b200 import clips
    spec = clips.CONFIGS[args.workload]
    t = spec.t if args.threshold is None else args.threshold
    budget = 150.0 / max(1, args.steps + args.warmup)
    Xs, desc = oracle_sample_plan(spec, t, budget)
    value, ms, tokens = run_oracle_steps(Xs, spec, t, args.steps, args.warmup)
    cores = O.threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(spec, t, len(Xs), 0, tokens),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def extensions_arm(args):
    """Times the extension entry points one by one on args.workload: every call on a clip that is cold in L2 (the
    calls rotate over args.clips distinct clips, together larger than L2), CUDA events on the launching stream.
    Bytes are the algorithmic ones of each operation; the fraction is against the measured copy rate."""
    import torch
    from paper_2605_07355_b200 import build as B
    from paper_2605_07355_b200 import clips
    import paper_2605_07355_b200 as P

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    B.build()
    P.lib()
    spec = clips.CONFIGS[args.workload]
    t = spec.t if args.threshold is None else args.threshold
    F, H, W, C, N = spec.F, spec.H, spec.W, spec.C, spec.H * spec.W
    row = C * spec.itemsize
    st = torch.cuda.Stream(device=dev)
    X, Q, comp, Ls = [], [], [], []
    for j in range(args.clips):
        Xn = clips.make_clip(spec, spec.seed + j)
        th = torch.from_numpy(Xn if spec.dtype == "f32" else Xn.view(np.int16))
        X.append((th if spec.dtype == "f32" else th.view(torch.bfloat16)).to(dev))
    with torch.cuda.stream(st):
        for x in X:
            Q.append(P.ttf_query(x, spec.r, t, stream=st))
            toks, cnt, _ = P.ttf_compress(x, spec.r, t, stream=st)
            L = int(cnt.item())
            Ls.append(L)
            comp.append(toks[:L].clone())
    torch.cuda.synchronize()
    Lm = float(np.mean(Ls))
    fused = F * N - Lm

    def timed(call):
        # warm pass (allocations, attribute set-up), then the pass over all clips captured in a CUDA graph, so that
        # the host cost of the Python calls stays outside the timed region
        with torch.cuda.stream(st):
            for j in range(len(X)):
                call(j)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            for j in range(len(X)):
                call(j)
        reps = max(3, args.steps // 10)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(st):
            g.replay()
            e0.record(st)
            for _ in range(reps):
                g.replay()
            e1.record(st)
        torch.cuda.synchronize()
        del g
        return e0.elapsed_time(e1) * 1e3 / (reps * len(X))

    pk_gbs, pk_src = peaks()
    out = {}

    def entry(name, us, nbytes, note):
        gbs = nbytes / us * 1e-3
        out[name] = {"us_per_clip": round(us, 2), "bytes_per_clip": int(nbytes), "achieved_gbs": round(gbs, 1),
                     "frac_of_copy_rate": round(gbs / pk_gbs, 3), "bytes": note}

    us = timed(lambda j: P.ttf_restore(comp[j], F, H, W, Q[j]["anchor"], Q[j]["keep"], Q[j]["dst"], stream=st))
    entry("ttf_restore", us, Lm * row + F * N * row + F * N * (1 + 4 + 4),
          "L' rows read, F*N rows written, keep + dst read, row_index written")
    us = timed(lambda j: P.ttf_compress_segment(X[j], spec.r, t, 0, stream=st))
    seg_keep = float(np.mean([int(P.ttf_compress_segment(x, spec.r, t, 0, stream=st)[1].item()) for x in X[:4]]))
    entry("ttf_compress_segment", us, F * N * row + seg_keep * (row + 12), "X read once, preserved rows and positions written")
    us = timed(lambda j: P.ttf_sim_histogram(Q[j]["best_sim"], Q[j]["anchor"], F, H, W, 256, stream=st))
    entry("ttf_sim_histogram", us, F * N * 4 + 256 * 4, "best_sim read, 256 counts written")
    us = timed(lambda j: P.ttf_compress_mean(X[j], spec.r, t, stream=st))
    entry("ttf_compress_mean", us, F * N * row + Lm * (row + 12) , "X read once, L' rows and positions written "
          "(the fused rows' second read for the means is traffic above that)")
    print(json.dumps({"extensions": out, "workload": workload_config(spec, t, args.clips, 1, F * N * args.clips)["workload"],
                      "clips": args.clips, "mean_L": Lm, "mean_fused": fused,
                      "peak_hbm_gbs": pk_gbs, "peak_source": pk_src,
                      "timing": "CUDA events around graph replays of one call per clip on one stream, clips together larger than L2"}))


def combine_ranks(ms_local: float, tokens_local: int, device=None):
    """Whole-job figures of a replica run: the slowest rank's time and the tokens of all ranks.  One clip never
    spans ranks, so this all-reduce of two scalars after the timed region is the only communication there is."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), int(tokens_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    n = torch.tensor([tokens_local], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), int(n.item())


def workload_config(spec, t, clips_per_step, streams, tokens_per_step, anchor="auto", graph=False, match_kernel="auto"):
    return {"workload": f"{spec.name}: F={spec.F} {spec.H}x{spec.W} C={spec.C} {spec.dtype} r={spec.r} t={t:.2f}",
            "generator": spec.family, "clips_per_step": clips_per_step, "tokens_per_step": tokens_per_step,
            "streams": streams, "anchor": anchor, "cuda_graph": graph, "match_kernel": match_kernel,
            "l2": "inputs rotate through a batch larger than L2; every clip starts cold in HBM"}


# ---------------------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    if args.impl == "reference":
        reference_arm(args)
        return
    if args.extensions:
        extensions_arm(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2605_07355_b200 import build as B
    from paper_2605_07355_b200 import accounting as A
    from paper_2605_07355_b200 import clips
    import paper_2605_07355_b200 as P

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if rank == 0:
        B.build()
    if world > 1:
        dist.barrier()
    P.lib()

    spec = clips.CONFIGS[args.workload]
    t = spec.t if args.threshold is None else args.threshold
    nclips = args.clips
    FN, C = spec.tokens, spec.C
    clip_bytes = FN * C * spec.itemsize
    tdtype = torch.float32 if spec.dtype == "f32" else torch.bfloat16

    # ---- inputs: pinned host copies (for the end-to-end leg) and device-resident copies -------------------
    host, devX = [], []
    for j in range(nclips):
        Xn = clips.make_clip(spec, spec.seed + 1000 * rank + j)
        th = torch.from_numpy(Xn if spec.dtype == "f32" else Xn.view(np.int16))
        th = (th if spec.dtype == "f32" else th.view(torch.bfloat16)).pin_memory()
        host.append(th)
        devX.append(th.to(dev, non_blocking=True))
    out_tok = [torch.empty((FN, C), dtype=tdtype, device=dev) for _ in range(nclips)]
    out_cnt = [torch.empty(1, dtype=torch.int32, device=dev) for _ in range(nclips)]
    out_pos = [torch.empty((FN, 3), dtype=torch.int32, device=dev) for _ in range(nclips)]
    torch.cuda.synchronize()

    nstreams = max(1, args.streams)
    main_stream = torch.cuda.Stream(device=dev)
    streams = [main_stream] if nstreams == 1 else [torch.cuda.Stream(device=dev) for _ in range(nstreams)]
    fork = torch.cuda.Event()
    joins = [torch.cuda.Event() for _ in streams]

    amode = {"auto": 0, "first": 1, "last": 2}[args.anchor]
    P.ttf_set_match_kernel({"auto": 0, "mma": 1, "tc": 2}[args.match_kernel])
    P.ttf_set_schedule(args.lanes)
    lanes = args.lanes if args.lanes > 0 else ("2, pipelined" if args.lanes == -1 and amode == 0 else 8)

    def step():
        if args.streams == 0:
            P.ttf_compress_batch(devX, spec.r, t, out_tok, out_cnt, out_pos, stream=main_stream, anchor_mode=amode)
            return
        if nstreams == 1:
            for j in range(nclips):
                P.ttf_compress(devX[j], spec.r, t, out_tok[j], out_cnt[j], out_pos[j], stream=main_stream,
                               anchor_mode=amode)
            return
        fork.record(main_stream)
        for s in streams:
            s.wait_event(fork)
        for j in range(nclips):
            P.ttf_compress(devX[j], spec.r, t, out_tok[j], out_cnt[j], out_pos[j], stream=streams[j % nstreams],
                           anchor_mode=amode)
        for s, ev in zip(streams, joins):
            ev.record(s)
            main_stream.wait_event(ev)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    launch_step = step
    for _ in range(max(3, args.warmup)):
        launch_step()
    barrier()
    use_graph = not args.no_graph
    if use_graph:
        # The step is launch-bound on the host (four kernels per clip, a few microseconds each to launch), so it
        # is captured once, C-ABI calls and all, and replayed.  Scratch was allocated by the warm-up calls.
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=main_stream):
            launch_step()

        def step():
            with torch.cuda.stream(main_stream):
                graph.replay()
        for _ in range(3):
            step()
        barrier()
    if args.ncu_range:
        torch.cuda.cudart().cudaProfilerStart()
        step()
        torch.cuda.synchronize()
        torch.cuda.cudart().cudaProfilerStop()
        print(json.dumps({"ncu_range": "one step", "workload": spec.name, "clips_per_step": nclips, "lanes": lanes,
                          "cuda_graph": use_graph, "counts": [int(c.item()) for c in out_cnt]}), flush=True)
        return
    counts = [int(c.item()) for c in out_cnt]
    rho = 1.0 - sum(counts) / float(nclips * FN)

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.05)

    # ---- timed region: exactly K steps, CUDA events on the launching stream (one event after every step, so
    # that the spread over the steps is known as well as the total) ------------------------------------------
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    w0 = time.perf_counter()
    marks[0].record(main_stream)
    for i in range(args.steps):
        step()
        marks[i + 1].record(main_stream)
    barrier()
    w1 = time.perf_counter()
    tokens_step = nclips * FN
    ms_total, tokens_all = combine_ranks(marks[0].elapsed_time(marks[-1]), tokens_step, dev)
    ms_step = ms_total / args.steps
    value = tokens_all / (ms_step * 1e-3)
    clips_per_s = value / FN
    per_step = sorted(marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps))
    pick = lambda q: per_step[min(len(per_step) - 1, int(q * len(per_step)))]
    step_ms = {"median": pick(0.5), "p10": pick(0.1), "p90": pick(0.9), "min": per_step[0], "max": per_step[-1]}

    # ---- latency of one clip when nothing else is in flight: the clips of the step one after the other on one
    # stream (captured like the step itself) ------------------------------------------------------------------
    lat_graph = torch.cuda.CUDAGraph()
    for j in range(min(nclips, 4)):
        P.ttf_compress(devX[j], spec.r, t, out_tok[j], out_cnt[j], out_pos[j], stream=main_stream, anchor_mode=amode)
    barrier()
    with torch.cuda.graph(lat_graph, stream=main_stream):
        for j in range(nclips):
            P.ttf_compress(devX[j], spec.r, t, out_tok[j], out_cnt[j], out_pos[j], stream=main_stream, anchor_mode=amode)
    l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(main_stream):
        lat_graph.replay()
        l0.record(main_stream)
        for _ in range(5):
            lat_graph.replay()
        l1.record(main_stream)
    barrier()
    latency_us = l0.elapsed_time(l1) * 1e3 / (5 * nclips)

    # ---- per-kernel durations at steady state: every kernel launched back to back for all clips of the step,
    # CUDA events (on the launching stream) around each group, divided by the clips; the batch is larger than L2,
    # so every launch finds its clip cold in HBM, as it does with several clips in flight --------------------
    sampler.stop()
    clocks = sampler.summary(w0, w1)
    kernel_ms = P.ttf_profile_stages(devX, spec.r, t, out_tok, out_cnt, out_pos, reps=min(args.steps, 20),
                                     stream=main_stream)
    # what the plainest read kernel takes on one clip, launched the same way: the floor for a kernel that reads a clip
    read_floor_us = 1e3 * P.ttf_profile_read_floor(devX, reps=min(args.steps, 20), stream=main_stream)
    torch.cuda.synchronize()
    launches_per_step = 4 * nclips      # sweep (or its stand-in for a fixed anchor), statistics or none, matching, gather
    if amode != 0:
        launches_per_step = 3 * nclips
    kern = {k: {"us_per_launch": 1e3 * v} for k, v in kernel_ms.items() if v > 0}
    tot = sum(kernel_ms.values())
    dominant = max(kern, key=lambda k: kernel_ms[k])
    peak_gbs, peak_kind = peaks()
    avg_count = sum(counts) / nclips
    kbytes = A.kernel_bytes(dominant, spec.F, spec.N, C, spec.itemsize, int(round(avg_count)))
    achieved = kbytes / (kern[dominant]["us_per_launch"] * 1e-6) / 1e9
    csrc = A.csrc_hash()
    traffic, traffic_note = stored_traffic(spec.name, dominant, csrc) if amode == 0 else (None, "no stored counters for this anchor rule")
    roofline = {"bound": "hbm", "kernel": dominant,
                "timed": "each kernel launched back to back for the clips of a step (cold in HBM), CUDA events around the group, / clips",
                "achieved": achieved, "peak": peak_gbs, "unit": "GB/s",
                "frac": achieved / peak_gbs, "peak_source": f"of {peak_kind}",
                "traffic": traffic, "traffic_note": traffic_note, "csrc_hash": csrc,
                "algorithmic_bytes_per_launch": kbytes,
                "read_floor": {"us_per_launch": round(read_floor_us, 3), "gbs": round(clip_bytes / read_floor_us * 1e-3, 1),
                               "what": "a plain coalesced read kernel over one clip (cold in HBM), launched back to back like "
                                       "the kernels above: what one launch that reads a clip once can reach"},
                "kernel_share": {k: kernel_ms[k] / tot for k in kern},
                "kernel_us": {k: round(kern[k]["us_per_launch"], 3) for k in kern},
                "kernel_frac": {k: A.kernel_bytes(k, spec.F, spec.N, C, spec.itemsize, int(round(avg_count)))
                                / (kern[k]["us_per_launch"] * 1e-6) / 1e9 / peak_gbs for k in kern}}
    bmin = A.pass_bytes(spec.F, spec.N, C, spec.itemsize, int(round(avg_count)))
    pass_gbs = bmin * nclips / (ms_step * 1e-3) / 1e9
    model = A.pipeline_dram_bytes_model(spec.F, spec.N, C, spec.itemsize, int(round(avg_count)),
                                        lanes if args.streams == 0 else nstreams, fixed_anchor=amode != 0)
    pass_roofline = {"bytes_per_clip": bmin, "achieved": pass_gbs, "unit": "GB/s", "frac_of_measured_copy": pass_gbs / peak_gbs,
                     "frac_of_8TBps": pass_gbs / 8000.0, "us_per_clip": ms_step * 1e3 / nclips,
                     "dram_bytes_per_clip_model": model,
                     "model_frac_of_measured_copy": model * nclips / (ms_step * 1e-3) / 1e9 / peak_gbs,
                     "latency_us_per_clip_one_stream": latency_us}

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region --------------------
    e2e = None
    if not args.no_e2e:
        # ttf_compress_host_batch: every step copies the clips in from pinned host memory, runs the pass and
        # copies L', the tokens and the positions back to pinned host memory, all inside the timed region
        h_tok = [torch.empty((FN, C), dtype=tdtype).pin_memory() for _ in range(nclips)]
        h_pos = [torch.empty((FN, 3), dtype=torch.int32).pin_memory() for _ in range(nclips)]
        P.ttf_compress_host_batch(host, spec.r, t, h_tok, h_pos)
        barrier()
        d2h = 0
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            _, Ls, _ = P.ttf_compress_host_batch(host, spec.r, t, h_tok, h_pos)
            d2h = sum(L * (C * spec.itemsize + 12) + 4 for L in Ls)
        barrier()
        dt = time.perf_counter() - t0
        dt_ms, tokens_e2e = combine_ranks(dt * 1e3, tokens_step * args.e2e_steps, dev)
        dt = dt_ms * 1e-3
        e2e = {"value": tokens_e2e / dt, "unit": UNIT,
               "h2d_bytes_per_step": nclips * clip_bytes, "d2h_bytes_per_step": d2h,
               "steps": args.e2e_steps, "api": "ttf_compress_host_batch (pinned host buffers; copies of consecutive clips overlap)"}

    # ---- the oracle on the host cores (rank 0, N = 1 only) ------------------------------------------------
    cpu = None
    if not args.no_cpu and world == 1 and rank == 0:
        from oracle import ttf_oracle as O
        Xs, desc = oracle_sample_plan(spec, t, args.cpu_seconds / 3.0)
        v, _, _ = run_oracle_steps(Xs, spec, t, 3, 0)
        cpu = {"value": v, "unit": UNIT, "cores": O.threads(), "kind": "oracle", "sample": desc + ", 3 steps"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": spec.dtype, "accumulate": "f32", "data": "synthetic",
            "config": workload_config(spec, t, nclips, f"{lanes} (library: ttf_compress_batch)" if args.streams == 0 else nstreams,
                                      tokens_step, args.anchor, use_graph, args.match_kernel),
            "step_ms": step_ms,
            "clips_per_s": clips_per_s, "rho": rho, "count_mean": avg_count,
            "roofline": roofline, "pass_roofline": pass_roofline, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches_per_step * args.steps), "gpu_launches_per_step": int(launches_per_step),
            "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
