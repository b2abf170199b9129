#!/usr/bin/env python
"""Benchmark of the tool-tracking hot path: frames/s over K concurrent streams, per-frame latency
distribution at a 16.7 ms frame period, and achieved fraction of the B200 roofline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--streams S]
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference     # the CPU oracle timed on the host cores

One "step" is one tick: the newest frame of every stream goes through the whole path
(preprocess, encoder, ConvLSTM step, postprocess, optional overlay).  `value` is whole-job
frames/s with the frames already resident in HBM, timed on the device with CUDA events on the
launching stream; `e2e` is the same metric through tt_submit_frames/tt_sync with pinned host
frames (host->device copies and the device->host result read inside the timed region).
Streams are independent, so with N GPUs every rank runs its own K streams (weak scaling, no
data-path collective); the reported time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "frames/s over K streams"
UNIT = "frames/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
FRAME_PERIOD_NS = 16_666_667


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"]))}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


KERNEL_SOURCES = {"convlstm": ["conv_tc.cu", "tc_ptx.cuh"], "enc1": ["conv_tc.cu", "tc_ptx.cuh"], "enc2": ["conv_tc.cu", "tc_ptx.cuh"],
                  "enc0": ["conv_first_tc.cu", "tc_ptx.cuh"], "preprocess": ["preprocess.cu"], "postprocess": ["postprocess.cu"],
                  "overlay": ["overlay.cu"]}


def kernel_source_hash(stage):
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES.get(stage, []):
        with open(os.path.join(ROOT, "paper_2402_04466_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(stage, workload, streams):
    """DRAM bytes per launch from the committed ncu capture, or None when there is none for this
    stage/workload or the kernel's source has changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    try:
        for line in open(path):
            f = line.split()
            if len(f) >= 5 and not line.startswith("#") and f[0] == stage and f[1] == workload and int(f[2]) == streams:
                return float(f[4]) if f[3] == kernel_source_hash(stage) else None
    except OSError:
        pass
    return None


def describe(wl, K):
    return (f"{wl.name}: K={K} concurrent streams, {wl.src_w}x{wl.src_h} uint8 RGB -> {wl.net_w}x{wl.net_h}, "
            f"encoder 3->{'->'.join(str(c) for c in wl.enc_cout)} (strides {list(wl.enc_stride)}), "
            f"ConvLSTM hidden {wl.hidden} on {wl.map_hw()[1]}x{wl.map_hw()[0]}, {wl.n_tools} tools, {wl.precision}"
            + (", overlay on" if wl.overlay else ""))


# ------------------------------------------------------------------------------ work model
def stage_work(wl, K):
    """Algorithmic bytes / flops of each stage for one tick of K stream-frames."""
    hm, wm = wl.map_hw()
    plane = hm * wm
    out = {}
    out["preprocess"] = {"bound": "hbm", "bytes": K * (3 * wl.src_w * wl.src_h + 12 * wl.net_w * wl.net_h)}
    h, w, cin = wl.net_h, wl.net_w, 3
    act_bytes = 2 if wl.precision == "bf16" else 4
    for l, (co, s) in enumerate(zip(wl.enc_cout, wl.enc_stride)):
        ho, wo = (h + 2 - 3) // s + 1, (w + 2 - 3) // s + 1
        flops = 2.0 * K * ho * wo * co * 9 * cin
        in_bytes = K * h * w * cin * (4 if l == 0 else act_bytes)
        out_bytes = K * ho * wo * co * act_bytes
        if l == 0 or wl.precision != "bf16":
            out[f"enc{l}"] = {"bound": "hbm" if l == 0 else "alu", "bytes": in_bytes + out_bytes, "flops": flops}
        else:
            out[f"enc{l}"] = {"bound": "tensor", "flops": flops, "bytes": in_bytes + out_bytes}
        h, w, cin = ho, wo, co
    ch = wl.hidden
    out["convlstm"] = {"bound": "tensor" if wl.precision == "bf16" else "alu",
                       "flops": 2.0 * K * plane * 4 * ch * 9 * (cin + ch),
                       "bytes": K * plane * (cin * act_bytes + ch * act_bytes + 8 * ch + 4 * ch + 2 * ch)}
    out["postprocess"] = {"bound": "hbm", "bytes": K * plane * (4 * ch + wl.n_tools * 9 + 1)}
    if wl.overlay:
        out["overlay"] = {"bound": "hbm", "bytes": K * (7 * wl.src_w * wl.src_h + plane)}
    return out


# ---------------------------------------------------------------------------- clock sampling
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        cmd = ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "25"]
        if uuid:
            cmd += ["-i", uuid]
        try:
            self.proc = subprocess.Popen(cmd, stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        rows = [r.strip().split(", ") for r in open(self.tmp.name).read().splitlines() if r.strip()]
        os.unlink(self.tmp.name)
        sm, reasons, smax = [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); smax = float(r[2])
            except ValueError:
                continue
            for name, v in zip(names, r[5:9]):
                if v.strip().lower().startswith("active"):
                    reasons.add(name)
        if sm:
            sm.sort()
            out.update({"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": smax, "reasons": sorted(reasons), "samples": len(sm)})
        return out


# ------------------------------------------------------------------------------ CPU oracle
def time_oracle(wl, budget_s=12.0, max_frames=8):
    """The oracle as it stands, on a bounded sample: whole stream-frames of this workload."""
    import oracle
    import tt_synth
    w = tt_synth.make_weights(wl)
    pipe = oracle.OraclePipeline(wl, w)
    n, t_total = 0, 0.0
    while n < max_frames and (n == 0 or t_total < budget_s):
        fr = tt_synth.make_frame(wl.frame_kind, wl.stream_seed(0), n, wl.src_w, wl.src_h)
        t0 = time.perf_counter()
        pipe.step(fr)
        t_total += time.perf_counter() - t0
        n += 1
    return {"value": n / t_total, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{n} stream-frames of {wl.name} (one stream, consecutive frames) in {t_total:.1f} s; "
                      "per-frame cost is independent of K, so K streams cost K times as much"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    import tt_synth
    wl = tt_synth.workload(args.workload)
    K = args.streams or wl.streams
    w = tt_synth.make_weights(wl)
    pipe = oracle.OraclePipeline(wl, w)
    frames = [tt_synth.make_frame(wl.frame_kind, wl.stream_seed(0), t, wl.src_w, wl.src_h) for t in range(4)]
    for i in range(args.warmup):
        t0 = time.perf_counter()
        pipe.step(frames[i % 4])
        if (time.perf_counter() - t0) * (args.steps + args.warmup - i) > 240 and i >= 0:
            break
    times, budget = [], 240.0
    for i in range(args.steps):
        t0 = time.perf_counter()
        pipe.step(frames[i % 4])
        times.append(time.perf_counter() - t0)
        if sum(times) > budget:
            break
    total = sum(times)
    value = len(times) / total
    sample = (f"each step = 1 stream-frame of {wl.name} through the CPU oracle ({oracle.num_threads()} host threads); "
              f"{len(times)} of {args.steps} requested steps fitted the time budget")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": 0, "steps": len(times),
            "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(wl, K), "note": "one stream-frame per step; oracle cost scales linearly in K"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


def paced_run(ctx, states, host_ring, K, R, n_frames):
    """Frames of all K streams arrive together every 16.667 ms (pinned host memory); latency of a tick =
    scheduled arrival -> tt_sync returned.  First and last 10 frames dropped (paper, Section VI)."""
    import ctypes as C

    import numpy as np

    from paper_2402_04466_b200 import binding
    from paper_2402_04466_b200.stats import latency_summary, trim_warmup
    try:
        os.sched_setaffinity(0, {sorted(os.sched_getaffinity(0))[-1]})
    except Exception:
        pass
    fr = (binding.tt_frame * K)()
    sts = (C.c_void_p * K)(*[s.value for s in states])
    res = (binding.tt_result * binding.TT_MAX_STREAMS)()
    lat_ms, gpu_ms, misses = [], [], 0
    t_start = time.perf_counter_ns() + 2_000_000
    for i in range(n_frames):
        arrival = t_start + i * FRAME_PERIOD_NS
        while time.perf_counter_ns() < arrival:
            pass
        for s in range(K):
            fr[s].data = host_ring[s][i % R].data_ptr()
            fr[s].on_device = 0
            fr[s].frame_index = i
            fr[s].arrival_ns = arrival
        st = ctx.submit_raw(K, fr, sts)
        st = st or ctx.sync_raw(res)
        done = time.perf_counter_ns()
        if st != 0:
            raise RuntimeError(f"paced run failed: {ctx.last_error()}")
        lat_ms.append((done - arrival) / 1e6)
        gpu_ms.append(res[0].gpu_ms)
        misses += int(done - arrival > FRAME_PERIOD_NS)
    latency = latency_summary(trim_warmup(lat_ms))
    latency.update({"streams": K, "frames_per_stream": n_frames, "frame_period_ms": FRAME_PERIOD_NS / 1e6,
                    "deadline_misses": misses, "gpu_ms_mean": float(np.mean(trim_warmup(gpu_ms))),
                    "definition": "scheduled arrival of the K frames -> tt_sync returned (pinned host frames, H2D inside)"})
    return latency


def staggered_run(ctx, states, host_ring, K, R, n_frames, window_ns, seed):
    """Unsynchronised arrivals: every stream has its own seeded phase inside the 16.667 ms period.  The batch
    planner (tt_sched_*) coalesces frames that arrive within `window_ns` into one tick; up to two ticks are
    in flight.  Latency of a frame = its own arrival -> its tick's results were read by tt_sync."""
    import ctypes as C

    import numpy as np

    import tt_synth
    from paper_2402_04466_b200 import binding
    from paper_2402_04466_b200.stats import latency_summary
    sched = binding.Scheduler(max_streams=K, window_ns=window_ns, deadline_ns=FRAME_PERIOD_NS, max_in_flight=2,
                              budget_fraction=0.5, tick_ms_base=0.1, tick_ms_per_stream=0.03)
    sids = [sched.admit() for _ in range(K)]
    phases = (tt_synth.uniform01(seed, 999, K) * FRAME_PERIOD_NS).astype(np.int64)
    pending = sorted((int(phases[k]) + i * FRAME_PERIOD_NS, k, i) for k in range(K) for i in range(n_frames))
    res = (binding.tt_result * binding.TT_MAX_STREAMS)()
    inflight, lat, sizes = [], [], []
    t0 = time.perf_counter_ns() + 2_000_000
    while True:
        now = time.perf_counter_ns() - t0
        while inflight and ctx.query():
            if ctx.sync_raw(res) != 0:
                raise RuntimeError(f"staggered run failed: {ctx.last_error()}")
            done = time.perf_counter_ns() - t0
            batch = inflight.pop(0)
            sched.complete(res[0].gpu_ms, done)
            lat.extend((fi, (done - arr) / 1e6) for _, fi, arr in batch)
        while pending and pending[0][0] <= now:
            t_arr, k, i = pending.pop(0)
            sched.arrive(sids[k], i, t_arr)
        batch, wake = sched.next(now)
        if batch:
            fr = (binding.tt_frame * len(batch))()
            sts = (C.c_void_p * len(batch))(*[states[s].value for s, _, _ in batch])
            for j, (s_, fi, arr) in enumerate(batch):
                fr[j].data = host_ring[s_][fi % R].data_ptr()
                fr[j].on_device = 0
                fr[j].frame_index = fi
                fr[j].arrival_ns = arr
            if ctx.submit_raw(len(batch), fr, sts) != 0:
                raise RuntimeError(f"staggered submit failed: {ctx.last_error()}")
            inflight.append(batch)
            sizes.append(len(batch))
        elif not pending and not inflight and wake == binding.Scheduler.NEVER:
            break
    kept = [l for fi, l in lat if 10 <= fi < n_frames - 10]
    out = latency_summary(kept)
    out.update(sched.stats())
    out.update({"streams": K, "frames_per_stream": n_frames, "window_ms": window_ns / 1e6, "mean_batch": float(np.mean(sizes)),
                "phases_ms": [round(float(p) / 1e6, 3) for p in phases],
                "definition": "own arrival of a frame -> tt_sync of its tick returned; arrivals staggered by a seeded phase per stream"})
    return out


# -------------------------------------------------------------------------------- GPU arm
def run_ours(args):
    import ctypes as C

    import numpy as np
    import torch
    import torch.distributed as dist

    import tt_synth
    from paper_2402_04466_b200 import binding
    from paper_2402_04466_b200.stats import latency_summary, trim_warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    wl = tt_synth.workload(args.workload)
    K = args.streams or wl.streams
    if args.overlay is not None:
        wl = wl.with_(overlay=bool(args.overlay))
    weights = tt_synth.make_weights(wl)
    stream = torch.cuda.Stream()
    cfg = binding.make_config(wl, max_streams=K, device=local_rank, cuda_stream=stream.cuda_stream)
    ctx = binding.Context(cfg, weights)
    states = [ctx.state_create() for _ in range(K)]

    # ring of distinct frames per stream (seeded; stream s of rank r uses seed index r*K + s)
    R = args.ring
    host_ring = [[torch.from_numpy(tt_synth.make_frame(wl.frame_kind, wl.stream_seed(rank * K + s), t, wl.src_w, wl.src_h)).pin_memory()
                  for t in range(R)] for s in range(K)]
    dev_ring = [[f.to(dev) for f in host_ring[s]] for s in range(K)]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    frame_bytes = wl.src_h * wl.src_pitch

    def tick(i, ring):
        ctx.submit_frames([ring[s][i % R] for s in range(K)], states, frame_index=i)
        return ctx.sync()

    def flush_l2(i):
        with torch.cuda.stream(stream):
            flush.fill_(i & 0xFF)

    for i in range(args.warmup):
        flush_l2(i)
        tick(i, dev_ring)

    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:
        pass
    sampler = ClockSampler(uuid) if rank == 0 else None
    launches0, _ = ctx.get_counters()

    # ---- timed region 1: device-resident frames, device time per tick from CUDA events
    barrier()
    step_ms = []
    for i in range(args.steps):
        flush_l2(i)
        res = tick(i, dev_ring)
        step_ms.append(res[0]["gpu_ms"])
    barrier()
    launches1, _ = ctx.get_counters()
    total_ms = float(sum(step_ms))

    # ---- the same K steps again with an event recorded after every stage (per-kernel durations for
    # the roofline figures; the extra event records cost a few percent, so `value` comes from above)
    ctx.set_profiling(True)
    stage_sum, prof_ms = {}, 0.0
    for i in range(args.steps):
        flush_l2(i)
        res = tick(i, dev_ring)
        prof_ms += res[0]["gpu_ms"]
        for k, v in ctx.get_stage_times().items():
            stage_sum[k] = stage_sum.get(k, 0.0) + v
    ctx.set_profiling(False)
    barrier()

    # ---- timed region 2: end to end through the public calls with pinned host frames.
    # (a) one tick at a time: submit -> sync, L2 flushed outside the timed part;
    # (b) software-pipelined, the way a throughput-oriented caller drives the API: tick i+1 is
    #     submitted before tick i is synced, so its host->device copy overlaps tick i's compute.
    #     The L2 flush stays in stream order between ticks and its time counts against the number.
    barrier()
    e2e_serial_s = 0.0
    for i in range(args.steps):
        flush_l2(i)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        tick(i, host_ring)
        e2e_serial_s += time.perf_counter() - t0
    barrier()
    t0 = time.perf_counter()
    flush_l2(0)
    ctx.submit_frames([host_ring[s][0] for s in range(K)], states, frame_index=0)
    for i in range(1, args.steps):
        flush_l2(i)
        ctx.submit_frames([host_ring[s][i % R] for s in range(K)], states, frame_index=i)
        ctx.sync()
    ctx.sync()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    barrier()
    clocks = sampler.stop() if sampler else None

    if world > 1:
        t = torch.tensor([total_ms, e2e_s, e2e_serial_s], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms, e2e_s, e2e_serial_s = float(t[0]), float(t[1]), float(t[2])

    # ---- paced latency run (rank 0 of a single-GPU job): frames arrive every 16.7 ms per stream
    latency = None
    if world == 1 and args.paced_frames > 0:
        for s in states:
            ctx.state_reset(s)
        latency = paced_run(ctx, states, host_ring, K, R, args.paced_frames)

    staggered = None
    if world == 1 and args.staggered_frames > 0:
        for s in states:
            ctx.state_reset(s)
        staggered = staggered_run(ctx, states, host_ring, K, R, args.staggered_frames, int(args.window_ms * 1e6), wl.seed)

    # ---- optional sweep over the number of streams (spec report: K = 1..8)
    sweep = None
    if world == 1 and args.sweep:
        sweep = []
        for Ks in [int(x) for x in args.sweep.split(",")]:
            wls = wl
            ctx_s = binding.Context(binding.make_config(wls, max_streams=Ks, device=local_rank, cuda_stream=stream.cuda_stream), weights)
            st_s = [ctx_s.state_create() for _ in range(Ks)]
            ring_h = [host_ring[s % K] for s in range(Ks)]
            ring_d = [dev_ring[s % K] for s in range(Ks)]
            ms = []
            for i in range(args.warmup + args.sweep_steps):
                flush_l2(i)
                ctx_s.submit_frames([ring_d[s][i % R] for s in range(Ks)], st_s, frame_index=i)
                r = ctx_s.sync()
                if i >= args.warmup:
                    ms.append(r[0]["gpu_ms"])
            ent = {"streams": Ks, "frames_per_s": Ks * len(ms) / (sum(ms) * 1e-3), "ms_per_tick": sum(ms) / len(ms)}
            if args.sweep_paced_frames > 0:
                for s_ in st_s:
                    ctx_s.state_reset(s_)
                lat = paced_run(ctx_s, st_s, ring_h, Ks, R, args.sweep_paced_frames)
                ent.update({k: lat[k] for k in ("p50_ms", "p99_ms", "max_ms", "spread_p99_p50_ms", "flatness_p90_p10_ms",
                                                "tail_p100_p95_ms", "deadline_misses", "gpu_ms_mean")})
            sweep.append(ent)
            ctx_s.destroy()

    if rank != 0:
        ctx.destroy()
        if world > 1:
            dist.destroy_process_group()
        return 0

    peaks, peak_kind = load_peaks()
    work = stage_work(wl, K)
    stages = {}
    for name, wk in work.items():
        if name not in stage_sum:
            continue
        ms = stage_sum[name] / args.steps
        ent = {"ms": ms, "bound": wk["bound"]}
        if wk["bound"] == "hbm":
            ent.update({"achieved": wk["bytes"] / (ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"})
        elif wk["bound"] == "tensor":
            ent.update({"achieved": wk["flops"] / (ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"})
        else:
            ent.update({"achieved": wk["flops"] / (ms * 1e-3) / 1e12, "peak": None, "unit": "TFLOP/s"})
        ent["frac"] = ent["achieved"] / ent["peak"] if ent.get("peak") else None
        stages[name] = ent
    dom = max(stages, key=lambda n: stages[n]["ms"])
    d = stages[dom]
    roofline = {"kernel": dom, "bound": d["bound"], "achieved": d["achieved"], "peak": d["peak"], "unit": d["unit"],
                "frac": d["frac"], "traffic": recorded_traffic(dom, wl.name.replace("-gain", ""), K), "peak_source": f"of {peak_kind} (burst figure)",
                "launch_ms": d["ms"]}

    cpu_baseline = time_oracle(wl.with_(overlay=False)) if (world == 1 and not args.no_cpu_baseline) else None
    n_frames = world * K * args.steps
    line = {
        "metric": METRIC, "value": n_frames / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "ms_per_step_with_stage_events": prof_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if wl.precision == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": describe(wl, K), "streams_per_gpu": K, "frame_ring": R,
                   "l2": "flushed between timed steps (256 MiB device write outside the timed events)",
                   "timing": "CUDA events on the launching stream around every tick, summed over the timed steps"},
        "e2e": {"value": n_frames / e2e_s, "unit": UNIT, "h2d_bytes_per_step": K * frame_bytes,
                "d2h_bytes_per_step": K * C.sizeof(binding.tt_result) + 4,
                "serial_value": n_frames / e2e_serial_s,
                "timing": "host clock, pinned host frames; value: two submits in flight (tick i+1 submitted before tick i is "
                          "synced), L2 flush between ticks included; serial_value: submit -> sync one tick at a time, "
                          "flush outside the timed part"},
        "gpu_launches": launches1 - launches0,
        "roofline": roofline, "stages": stages, "clocks": clocks,
    }
    if latency is not None:
        line["latency"] = latency
    if staggered is not None:
        line["latency_staggered"] = staggered
    if sweep is not None:
        line["sweep"] = sweep
    if cpu_baseline is not None:
        line["cpu_baseline"] = cpu_baseline
    print(json.dumps(line))
    ctx.destroy()
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", help="cfg0..cfg4 (optionally with -gain)")
    ap.add_argument("--streams", type=int, default=0, help="streams per GPU (default: the workload's)")
    ap.add_argument("--overlay", type=int, default=None)
    ap.add_argument("--ring", type=int, default=8, help="distinct frames per stream, reused cyclically")
    ap.add_argument("--paced-frames", type=int, default=600, help="frames per stream of the paced latency run (0: skip)")
    ap.add_argument("--staggered-frames", type=int, default=0,
                    help="frames per stream of the unsynchronised-arrival run through the batch planner (0: skip)")
    ap.add_argument("--window-ms", type=float, default=1.0, help="coalescing window of the batch planner")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", default="", help="comma-separated stream counts to measure in addition, e.g. 1,2,3,4,5,6,7,8")
    ap.add_argument("--sweep-steps", type=int, default=100)
    ap.add_argument("--sweep-paced-frames", type=int, default=200)
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
