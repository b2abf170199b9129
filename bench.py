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
# plain fp32 arithmetic: 148 multiprocessors x 128 FMA lanes x 2 flops at the 1965 MHz maximum clock (derived, not measured)
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12
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
                  "enc0": ["conv_first_tc.cu", "tc_ptx.cuh", "pre_math.cuh"], "preprocess": ["preprocess.cu", "pre_math.cuh"], "postprocess": ["post_tc.cu", "tc_ptx.cuh"],
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
    # on the bf16 path the heads run on the tensor cores from the bf16 copy of h' when the hidden width is a
    # multiple of 64 and the map has at least 128 pixels; the ConvLSTM then writes no fp32 copy of h'
    heads_bf16 = wl.precision == "bf16" and ch % 64 == 0 and ch <= 512 and plane >= 128
    if getattr(wl, "recurrent", True):
        out["convlstm"] = {"bound": "tensor" if wl.precision == "bf16" else "alu",
                           "flops": 2.0 * K * plane * 4 * ch * 9 * (cin + ch),
                           "bytes": K * plane * (cin * act_bytes + ch * act_bytes + 8 * ch + (0 if heads_bf16 else 4 * ch) + 2 * ch)}
    out["postprocess"] = {"bound": "hbm", "bytes": K * plane * ((2 if heads_bf16 else 4) * ch + wl.n_tools * 9 + 1)}
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
def cpu_model():
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def time_oracle(wl, budget_s=12.0, max_frames=8, single_thread_frames=1):
    """The oracle as it stands, on a bounded sample: whole stream-frames of this workload, first on all
    host threads the oracle uses, then on one thread."""
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
    threads = oracle.num_threads()
    out = {"value": n / t_total, "unit": UNIT, "cores": threads, "kind": "oracle", "cpu_model": cpu_model(),
           "host_cpus": os.cpu_count(),
           "sample": f"{n} stream-frames of {wl.name} (one stream, consecutive frames) in {t_total:.1f} s; "
                     "per-frame cost is independent of K, so K streams cost K times as much"}
    if single_thread_frames > 0:
        oracle.set_threads(1)
        try:
            t1 = 0.0
            for i in range(single_thread_frames):
                fr = tt_synth.make_frame(wl.frame_kind, wl.stream_seed(0), n + i, wl.src_w, wl.src_h)
                t0 = time.perf_counter()
                pipe.step(fr)
                t1 += time.perf_counter() - t0
        finally:
            oracle.set_threads(threads)
        out["single_thread"] = {"value": single_thread_frames / t1, "unit": UNIT, "cores": 1,
                                "sample": f"{single_thread_frames} stream-frame(s) of {wl.name} in {t1:.1f} s"}
    return out


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
            "config": {"workload": describe(wl, K)},
            "note": "one stream-frame per step; oracle cost scales linearly in K",
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample,
                             "cpu_model": cpu_model()},
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
    pinned_cpu = None
    try:
        pinned_cpu = sorted(os.sched_getaffinity(0))[-1]
        os.sched_setaffinity(0, {pinned_cpu})
    except Exception:
        pinned_cpu = None
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
                    "deadline_misses": misses, "gpu_ms_mean": float(np.mean(trim_warmup(gpu_ms))), "pacing_thread_cpu": pinned_cpu,
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
    # Admission control under over-subscription (paper, Section IV-A): a planner that has seen this run's tick
    # times is given a budget of 1.5 x the observed one-stream tick and admits streams until one is refused.
    tick1 = sched.predict_ms(1)
    tight = binding.Scheduler(max_streams=binding.TT_MAX_STREAMS, window_ns=window_ns, deadline_ns=FRAME_PERIOD_NS, max_in_flight=2,
                              budget_fraction=min(1.0, 1.5 * tick1 / (FRAME_PERIOD_NS / 1e6)), tick_ms_base=0.8 * tick1,
                              tick_ms_per_stream=0.2 * tick1)
    admitted = 0
    try:
        while admitted < binding.TT_MAX_STREAMS:
            tight.admit()
            admitted += 1
    except binding.TTError as e:
        if e.status != 5:
            raise
    out["admission_demo"] = {"budget_ms": 1.5 * tick1, "tick_ms_model": f"{0.8 * tick1:.4f} + {0.2 * tick1:.4f} per stream (from this run's one-stream ticks)",
                             "streams_admitted": admitted, "refused_at": admitted + 1 if admitted < binding.TT_MAX_STREAMS else None}
    out.update({"streams": K, "frames_per_stream": n_frames, "window_ms": window_ns / 1e6, "mean_batch": float(np.mean(sizes)),
                "phases_ms": [round(float(p) / 1e6, 3) for p in phases],
                "definition": "own arrival of a frame -> tt_sync of its tick returned; arrivals staggered by a seeded phase per stream"})
    return out


# ------------------------------------------------- studies beyond the headline (run on request)
def paced_multi(parts, n_frames, before_tick=None):
    """Several contexts driven in lock step: every 16.667 ms the frames of all parts arrive together, every part is
    submitted (each on its own context), then every part is synced in turn.  parts: list of dicts with ctx, states,
    host_ring (pinned), K, R.  Returns per part the latency summary (arrival -> that part's tt_sync returned) and,
    under "all", arrival -> the last part returned.  before_tick(i) runs right after the arrival of frame i."""
    import ctypes as C

    from paper_2402_04466_b200 import binding
    from paper_2402_04466_b200.stats import latency_summary, trim_warmup
    try:
        os.sched_setaffinity(0, {sorted(os.sched_getaffinity(0))[-1]})
    except Exception:
        pass
    for p in parts:
        p["fr"] = (binding.tt_frame * p["K"])()
        p["sts"] = (C.c_void_p * p["K"])(*[s.value for s in p["states"]])
        p["res"] = (binding.tt_result * binding.TT_MAX_STREAMS)()
        p["lat"] = []
    lat_all = []
    t_start = time.perf_counter_ns() + 2_000_000
    for i in range(n_frames):
        arrival = t_start + i * FRAME_PERIOD_NS
        while time.perf_counter_ns() < arrival:
            pass
        if before_tick is not None:
            before_tick(i)
        for p in parts:
            for s in range(p["K"]):
                p["fr"][s].data = p["host_ring"][s][i % p["R"]].data_ptr()
                p["fr"][s].on_device = 0
                p["fr"][s].frame_index = i
                p["fr"][s].arrival_ns = arrival
            if p["ctx"].submit_raw(p["K"], p["fr"], p["sts"]) != 0:
                raise RuntimeError(p["ctx"].last_error())
        for p in parts:
            if p["ctx"].sync_raw(p["res"]) != 0:
                raise RuntimeError(p["ctx"].last_error())
            p["lat"].append((time.perf_counter_ns() - arrival) / 1e6)
        lat_all.append((time.perf_counter_ns() - arrival) / 1e6)
    keys = ("mean_ms", "std_ms", "p50_ms", "p99_ms", "max_ms", "tail_p100_p95_ms", "flatness_p90_p10_ms")
    out = {"all": {k: latency_summary(trim_warmup(lat_all))[k] for k in keys}}
    for j, p in enumerate(parts):
        out[p.get("name", f"part{j}")] = {k: latency_summary(trim_warmup(p["lat"]))[k] for k in keys}
    return out


def render_study(args):
    """Single-GPU isolation of the visualisation load (the paper's Section VIII future work, asked with CUDA only).
    While tick i is computed, the multi-layer render of tick i-1's masks runs on a second stream, either
    time-shared (spread over every multiprocessor) or carved out (a few looping blocks on multiprocessors the
    inference context leaves free).  Per-frame latency of the inference ticks for K = 1..6."""
    import numpy as np
    import torch

    import tt_synth
    from paper_2402_04466_b200 import binding
    dev = torch.device("cuda", 0)
    wl = tt_synth.workload("cfg3").with_(overlay=False)
    R, carve = args.ring, args.carve_sms
    rstream = torch.cuda.Stream()
    rows = []
    for K in [int(x) for x in args.study_streams.split(",")]:
        frames = [[torch.from_numpy(tt_synth.make_frame(wl.frame_kind, wl.stream_seed(s), t, wl.src_w, wl.src_h)) for t in range(R)]
                  for s in range(K)]
        host_ring = [[f.pin_memory() for f in fs] for fs in frames]
        stacked = [torch.stack([frames[s][t].reshape(-1) for s in range(K)]).to(dev) for t in range(R)]   # [K][bytes] per ring index
        out_buf = torch.empty((K, wl.src_h, wl.src_w, 4), dtype=torch.uint8, device=dev)
        hm, wm = wl.map_hw()
        for mode in ("none", "time-shared", "carved-out"):
            stream = torch.cuda.Stream()
            cfg = binding.make_config(wl, max_streams=K, cuda_stream=stream.cuda_stream, reserved_sms=carve if mode == "carved-out" else 0)
            ctx = binding.Context(cfg, tt_synth.make_weights(wl))
            part = {"name": "inference", "ctx": ctx, "states": [ctx.state_create() for _ in range(K)], "host_ring": host_ring, "K": K, "R": R}
            state = {"masks": None}
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            render_ms = []

            def before_tick(i):
                # the masks of the previous tick are rendered while this tick is computed
                if mode == "none" or i == 0:
                    return
                res0 = part["res"][0]
                masks = binding.device_tensor(res0.masks_dev, (K, wl.n_tools, hm, wm), np.uint8)
                timed = (i % 16 == 1)
                with torch.cuda.stream(rstream):
                    if timed:
                        ev0.record()
                    binding.render_layers(stacked[(i - 1) % R], wl.src_w, wl.src_h, wl.src_pitch, masks, wl.palette, args.render_layers,
                                          carve_ctas=carve if mode == "carved-out" else 0, stream=rstream, out=out_buf)
                    if timed:
                        ev1.record()
                        state["pending"] = True

            def harvest():
                if state.get("pending"):
                    ev1.synchronize()
                    render_ms.append(ev0.elapsed_time(ev1))
                    state["pending"] = False

            # harvest the timed render of the previous period right at the next arrival (it has long finished)
            def hook(i):
                harvest()
                before_tick(i)

            lat = paced_multi([part], args.study_frames, before_tick=hook)
            torch.cuda.synchronize()
            harvest()
            ent = {"streams": K, "mode": mode, **lat["inference"]}
            if render_ms:
                ent["render_ms_mean"] = sum(render_ms) / len(render_ms)
                ent["render_ms_max"] = max(render_ms)
            rows.append(ent)
            ctx.destroy()
    print(json.dumps({"study": "render isolation", "workload": describe(wl, 0).replace("K=0 ", ""), "render_layers": args.render_layers,
                      "carved_out_sms": carve, "frames_per_stream": args.study_frames, "rows": rows}))
    return 0


def hetero_study(args):
    """Two different models on one GPU (the paper's heterogeneous experiment, Section VI, Table II): the recurrent
    tool-tracking model and a feed-forward segmentation model, alone and together (each context on its own CUDA
    stream, both submitted every period)."""
    import torch

    import tt_synth
    from paper_2402_04466_b200 import binding
    dev = torch.device("cuda", 0)
    R = args.ring
    specs = {"tool-tracking (recurrent)": (tt_synth.workload("cfg2"), args.hetero_k),
             "segmentation (feed-forward)": (tt_synth.workload("cfg2-ff"), args.hetero_k)}

    def build(name, shared_stream=None):
        wl, K = specs[name]
        stream = shared_stream or torch.cuda.Stream()
        ctx = binding.Context(binding.make_config(wl, max_streams=K, cuda_stream=stream.cuda_stream), tt_synth.make_weights(wl))
        host_ring = [[torch.from_numpy(tt_synth.make_frame(wl.frame_kind, wl.stream_seed(s), t, wl.src_w, wl.src_h)).pin_memory()
                      for t in range(R)] for s in range(K)]
        return {"name": name, "ctx": ctx, "states": [ctx.state_create() for _ in range(K)], "host_ring": host_ring, "K": K, "R": R,
                "_stream": stream}

    rows = []
    for name in specs:
        p = build(name)
        rows.append({"setup": "alone", **{name: paced_multi([p], args.study_frames)[name]}})
        p["ctx"].destroy()
    parts = [build(n) for n in specs]
    lat = paced_multi(parts, args.study_frames)
    rows.append({"setup": "together, one CUDA stream per model", **lat})
    for p in parts:
        p["ctx"].destroy()
    one = torch.cuda.Stream()
    parts = [build(n, one) for n in specs]
    lat = paced_multi(parts, args.study_frames)
    rows.append({"setup": "together, both models on one CUDA stream (serialised)", **lat})
    for p in parts:
        p["ctx"].destroy()
    print(json.dumps({"study": "heterogeneous models", "streams_per_model": args.hetero_k, "frames_per_stream": args.study_frames,
                      "models": {n: describe(w, k) for n, (w, k) in specs.items()}, "rows": rows}))
    return 0


def multi_model_study(args):
    """Three models per frame (the paper's Multi-AI application, Section III-B): three feed-forward encoder/head sets
    with different weights read the same frame; latency = arrival -> all three results on the host."""
    import torch

    import tt_synth
    from paper_2402_04466_b200 import binding
    R = args.ring
    base = tt_synth.workload("cfg2-ff")
    wls = [base.with_(name=f"model{j}", seed=base.seed + 31 * (j + 1)) for j in range(3)]
    host_ring = [[torch.from_numpy(tt_synth.make_frame(base.frame_kind, base.stream_seed(0), t, base.src_w, base.src_h)).pin_memory()
                  for t in range(R)]]

    def build(wl, stream):
        ctx = binding.Context(binding.make_config(wl, max_streams=1, cuda_stream=stream.cuda_stream), tt_synth.make_weights(wl))
        return {"name": wl.name, "ctx": ctx, "states": [ctx.state_create()], "host_ring": host_ring, "K": 1, "R": R}

    rows = []
    for setup, streams in (("three CUDA streams (concurrent branches)", [torch.cuda.Stream() for _ in range(3)]),
                           ("one CUDA stream (serialised)", [torch.cuda.Stream()] * 3)):
        parts = [build(w, s) for w, s in zip(wls, streams)]
        lat = paced_multi(parts, args.study_frames)
        rows.append({"setup": setup, **lat})
        for p in parts:
            p["ctx"].destroy()
    p = build(wls[0], torch.cuda.Stream())
    rows.append({"setup": "one model alone", **paced_multi([p], args.study_frames)})
    p["ctx"].destroy()
    print(json.dumps({"study": "three models per frame", "model": describe(base, 1), "frames_per_stream": args.study_frames, "rows": rows}))
    return 0


# -------------------------------------------------------------------------------- GPU arm
def stage_table(wl, K, stage_sum, steps, peaks):
    """Per-stage device time, achieved rate and fraction of the roof that bounds the stage."""
    stages = {}
    for name, wk in stage_work(wl, K).items():
        if name not in stage_sum:
            continue
        ms = stage_sum[name] / steps
        ent = {"ms": ms, "bound": wk["bound"]}
        if wk["bound"] == "hbm":
            ent.update({"achieved": wk["bytes"] / (ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"})
        elif wk["bound"] == "tensor":
            ent.update({"achieved": wk["flops"] / (ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"})
            ent["frac_of_sustained"] = ent["achieved"] / peaks["bf16_tflops_sustained"]
        else:
            ent.update({"achieved": wk["flops"] / (ms * 1e-3) / 1e12, "peak": FP32_ALU_TFLOPS, "unit": "TFLOP/s",
                        "peak_source": "derived: 148 SMs x 128 fp32 FMA lanes x 2 x 1.965 GHz (not measured)"})
        ent["frac"] = ent["achieved"] / ent["peak"]
        stages[name] = ent
    return stages


class Rig:
    """One context with K streams of a workload, its frame rings and the L2 flush buffer."""

    def __init__(self, wl, K, dev, local_rank, stream, ring, stream_ids, flush, host_frames=True):
        import torch

        import tt_synth
        from paper_2402_04466_b200 import binding
        self.wl, self.K, self.R, self.stream, self.flush = wl, K, ring, stream, flush
        self.weights = tt_synth.make_weights(wl)
        self.ctx = binding.Context(binding.make_config(wl, max_streams=K, device=local_rank, cuda_stream=stream.cuda_stream), self.weights)
        self.states = [self.ctx.state_create() for _ in range(K)]
        frames = [[torch.from_numpy(tt_synth.make_frame(wl.frame_kind, wl.stream_seed(sid), t, wl.src_w, wl.src_h)) for t in range(ring)]
                  for sid in stream_ids]
        self.host_ring = [[f.pin_memory() for f in fs] for fs in frames] if host_frames else None
        self.dev_ring = [[f.to(dev) for f in fs] for fs in frames]
        self.n_submits = 0
        self.settle()

    def settle(self):
        """Part of set-up, before any warm-up or timed step: the library captures one CUDA graph per (submit slot,
        frame buffer set, state ping-pong half) the first time each combination occurs, which takes host time inside
        that tick.  A ring of R device buffers meets lcm(slots, R, 2) combinations; run through all of them once."""
        import math

        from paper_2402_04466_b200 import binding
        for i in range(math.lcm(binding.TT_MAX_IN_FLIGHT, self.R, 2) + 1):
            self.tick(i, self.dev_ring)
        if self.host_ring is not None:      # host frames pass through the slot's staging buffer: slots x halves
            for i in range(math.lcm(binding.TT_MAX_IN_FLIGHT, 2) + 1):
                self.tick(i, self.host_ring)

    def flush_l2(self, i):
        import torch
        with torch.cuda.stream(self.stream):
            self.flush.fill_(i & 0xFF)

    def submit(self, i, ring, K=None):
        """Submit one tick.  The ring entry follows the context's own count of submits, not the caller's step index:
        submit slot, state ping-pong half and frame buffer set then stay in step, and a context only ever meets the
        lcm(slots, R, 2) graph keys it ran through while it was set up."""
        K = K or self.K
        self.ctx.submit_frames([ring[s][self.n_submits % self.R] for s in range(K)], self.states[:K], frame_index=i)
        self.n_submits += 1

    def tick(self, i, ring, K=None):
        self.submit(i, ring, K)
        return self.ctx.sync()

    def timed_ticks(self, steps, warmup):
        """-> summed device time (ms) of `steps` ticks on device-resident frames, L2 flushed before each."""
        for i in range(warmup):
            self.flush_l2(i)
            self.tick(i, self.dev_ring)
        ms = []
        for i in range(steps):
            self.flush_l2(i)
            ms.append(self.tick(i, self.dev_ring)[0]["gpu_ms"])
        return ms

    def stage_ticks(self, steps):
        """The same ticks with an event recorded after every stage -> summed stage times, summed tick time."""
        self.ctx.set_profiling(True)
        stage_sum, prof_ms = {}, 0.0
        for i in range(steps):
            self.flush_l2(i)
            res = self.tick(i, self.dev_ring)
            prof_ms += res[0]["gpu_ms"]
            for k, v in self.ctx.get_stage_times().items():
                stage_sum[k] = stage_sum.get(k, 0.0) + v
        self.ctx.set_profiling(False)
        return stage_sum, prof_ms

    def reset(self):
        for s in self.states:
            self.ctx.state_reset(s)

    def destroy(self):
        self.ctx.destroy()


def stream_sweep(rig_of, counts, steps, warmup, paced_frames):
    """frames/s and paced latency for several stream counts; rig_of(K) -> a Rig with at least K streams' frames."""
    out = []
    for Ks in counts:
        rig = rig_of(Ks)
        ms = rig.timed_ticks(steps, warmup)
        ent = {"streams": Ks, "frames_per_s": Ks * len(ms) / (sum(ms) * 1e-3), "ms_per_tick": sum(ms) / len(ms)}
        if paced_frames > 0:
            rig.reset()
            lat = paced_run(rig.ctx, rig.states, rig.host_ring, Ks, rig.R, paced_frames)
            ent.update({k: lat[k] for k in ("p50_ms", "p99_ms", "max_ms", "spread_p99_p50_ms", "flatness_p90_p10_ms",
                                            "tail_p100_p95_ms", "deadline_misses", "gpu_ms_mean")})
        out.append(ent)
        rig.destroy()
    return out


def run_ours(args):
    import ctypes as C

    import torch
    import torch.distributed as dist

    import tt_synth
    from paper_2402_04466_b200 import binding, sharding

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
    stream = torch.cuda.Stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    # Streams are independent problems: the world*K streams of the job are dealt round-robin to the ranks
    # (stream s lives on rank s mod world), each rank runs its K streams, nothing is exchanged on the GPU.
    my_streams = sharding.assign_streams(world * K, world)[rank]
    R = args.ring
    rig = Rig(wl, K, dev, local_rank, stream, R, my_streams, flush)
    ctx, states, host_ring, dev_ring = rig.ctx, rig.states, rig.host_ring, rig.dev_ring
    frame_bytes = wl.src_h * wl.src_pitch

    for i in range(args.warmup):
        rig.flush_l2(i)
        rig.tick(i, dev_ring)

    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:
        pass
    sampler = ClockSampler(uuid) if rank == 0 else None
    launches0, _ = ctx.get_counters()

    # ---- timed region 1: device-resident frames, device time per tick from CUDA events
    barrier()
    step_ms = rig.timed_ticks(args.steps, 0)
    barrier()
    launches1, _ = ctx.get_counters()
    total_ms = float(sum(step_ms))

    # ---- the same K steps again with an event recorded after every stage (per-kernel durations for
    # the roofline figures; the extra event records cost a few percent, so `value` comes from above)
    stage_sum, prof_ms = rig.stage_ticks(args.steps)
    barrier()

    # ---- timed region 2: end to end through the public calls with pinned host frames.
    # (a) one tick at a time: submit -> sync, L2 flushed outside the timed part;
    # (b) software-pipelined, the way a throughput-oriented caller drives the API: tick i+1 is
    #     submitted before tick i is synced, so its host->device copy overlaps tick i's compute.
    #     Once without any flush (every step's input crosses PCIe from host memory, so no cache can
    #     hold it; weights and activations stay where a running service would have them), once with
    #     the 256 MiB flush write in stream order between ticks, whose time then counts against the number.
    barrier()
    e2e_serial_s = 0.0
    for i in range(args.steps):
        rig.flush_l2(i)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        rig.tick(i, host_ring)
        e2e_serial_s += time.perf_counter() - t0
    barrier()

    def pipelined(with_flush):
        depth = binding.TT_MAX_IN_FLIGHT       # submits kept in flight: tick i + depth - 1 is submitted before tick i is synced
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        last = None
        for i in range(args.steps):
            if with_flush:
                rig.flush_l2(i)
            rig.submit(i, host_ring)
            if i >= depth - 1:
                last = ctx.sync()
        for _ in range(min(depth - 1, args.steps)):
            last = ctx.sync()
        torch.cuda.synchronize()
        return time.perf_counter() - t0, last

    e2e_s, last_results = pipelined(False)
    barrier()
    e2e_flush_s, _ = pipelined(True)
    barrier()

    total_ms, e2e_s, e2e_serial_s, e2e_flush_s = sharding.max_over_ranks([total_ms, e2e_s, e2e_serial_s, e2e_flush_s], world, device=dev)
    # host-side gather of the small per-frame result records of the last tick (the only cross-rank data)
    local = {sid: {"conf": [float(v) for v in r["conf"]], "count": [int(v) for v in r["count"]]} for sid, r in zip(my_streams, last_results)}
    gathered = sharding.gather_results(local, world)
    if len(gathered) != world * K:
        raise RuntimeError(f"gathered {len(gathered)} result records, expected {world * K}")

    # ---- paced latency run (rank 0 of a single-GPU job): frames arrive every 16.7 ms per stream
    latency = None
    if world == 1 and args.paced_frames > 0:
        rig.reset()
        latency = paced_run(ctx, states, host_ring, K, R, args.paced_frames)

    staggered = None
    if world == 1 and args.staggered_frames > 0:
        rig.reset()
        staggered = staggered_run(ctx, states, host_ring, K, R, args.staggered_frames, int(args.window_ms * 1e6), wl.seed)

    # the sampler covers the timed regions and the paced runs (a 20-step timed region alone lasts a few ms)
    clocks_main = sampler.stop() if sampler else None

    # ---- optional sweep over the number of streams of this workload
    sweep = None
    if world == 1 and args.sweep:
        counts = [int(x) for x in args.sweep.split(",")]
        sweep = stream_sweep(lambda Ks: Rig(wl, Ks, dev, local_rank, stream, R, [my_streams[s % K] for s in range(Ks)], flush),
                             counts, args.sweep_steps, args.warmup, args.sweep_paced_frames)

    peaks, peak_kind = load_peaks()

    # ---- the configuration the roofline targets are stated on (scale sweep, K = 8) and the stream-count
    # sweeps of both sizes, in the same process
    target = None
    if world == 1 and args.target_steps > 0 and not (wl.name == "cfg4" and K == 8):
        sampler_t = ClockSampler(uuid)
        wt = tt_synth.workload("cfg4")
        Kt = wt.streams
        rig_t = Rig(wt, Kt, dev, local_rank, stream, 2, [s for s in range(Kt)], flush, host_frames=True)
        ms_t = rig_t.timed_ticks(args.target_steps, args.warmup)
        stage_t, prof_t = rig_t.stage_ticks(args.target_steps)
        stages_t = stage_table(wt, Kt, stage_t, args.target_steps, peaks)
        target = {"workload": describe(wt, Kt), "steps": args.target_steps, "warmup": args.warmup,
                  "ms_per_step": sum(ms_t) / len(ms_t), "value": Kt * len(ms_t) / (sum(ms_t) * 1e-3), "unit": UNIT,
                  "ms_per_step_with_stage_events": prof_t / args.target_steps, "stages": stages_t,
                  "peaks": "tensor stages: frac against the measured burst bf16 peak, frac_of_sustained against the sustained one "
                           "(the tick runs under the power cap); hbm stages against the measured copy bandwidth"}
        if args.target_sweeps:
            rig_t.reset()
            sw4 = []
            for Ks in (1, 2, 4, 8):
                # one context sized for 8 streams serves every K: a tick of the first Ks streams
                ms = []
                for i in range(args.warmup + args.target_steps):
                    rig_t.flush_l2(i)
                    r = rig_t.tick(i, rig_t.dev_ring, Ks)
                    if i >= args.warmup:
                        ms.append(r[0]["gpu_ms"])
                rig_t.reset()
                lat = paced_run(rig_t.ctx, rig_t.states[:Ks], rig_t.host_ring, Ks, rig_t.R, args.target_paced_frames)
                sw4.append({"streams": Ks, "frames_per_s": Ks * len(ms) / (sum(ms) * 1e-3), "ms_per_tick": sum(ms) / len(ms),
                            "p50_ms": lat["p50_ms"], "p99_ms": lat["p99_ms"], "max_ms": lat["max_ms"],
                            "flatness_p90_p10_ms": lat["flatness_p90_p10_ms"], "deadline_misses": lat["deadline_misses"]})
            target["sweep_cfg4"] = sw4
        rig_t.destroy()
        if args.target_sweeps:
            sw2 = []
            w2 = tt_synth.workload("cfg2")
            rig_2 = Rig(w2, 8, dev, local_rank, stream, R, list(range(8)), flush)
            for Ks in range(1, 9):
                ms = []
                for i in range(args.warmup + 3 * args.target_steps):
                    rig_2.flush_l2(i)
                    r = rig_2.tick(i, rig_2.dev_ring, Ks)
                    if i >= args.warmup:
                        ms.append(r[0]["gpu_ms"])
                rig_2.reset()
                lat = paced_run(rig_2.ctx, rig_2.states[:Ks], rig_2.host_ring, Ks, rig_2.R, args.target_paced_frames)
                sw2.append({"streams": Ks, "frames_per_s": Ks * len(ms) / (sum(ms) * 1e-3), "ms_per_tick": sum(ms) / len(ms),
                            "p50_ms": lat["p50_ms"], "p99_ms": lat["p99_ms"], "max_ms": lat["max_ms"],
                            "flatness_p90_p10_ms": lat["flatness_p90_p10_ms"], "deadline_misses": lat["deadline_misses"]})
            rig_2.destroy()
            target["sweep_cfg2"] = sw2
        target["clocks"] = sampler_t.stop()

    if rank != 0:
        ctx.destroy()
        if world > 1:
            dist.destroy_process_group()
        return 0

    stages = stage_table(wl, K, stage_sum, args.steps, peaks)
    dom = max(stages, key=lambda n: stages[n]["ms"])
    d = stages[dom]
    roofline = {"kernel": dom, "bound": d["bound"], "achieved": d["achieved"], "peak": d["peak"], "unit": d["unit"],
                "frac": d["frac"], "traffic": recorded_traffic(dom, wl.name.replace("-gain", ""), K), "peak_source": f"of {peak_kind} (burst figure)",
                "launch_ms": d["ms"]}
    if "frac_of_sustained" in d:
        roofline["frac_of_sustained"] = d["frac_of_sustained"]

    cpu_baseline = time_oracle(wl.with_(overlay=False)) if (world == 1 and not args.no_cpu_baseline) else None
    n_frames = world * K * args.steps
    line = {
        "metric": METRIC, "value": n_frames / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "ms_per_step_with_stage_events": prof_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if wl.precision == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": describe(wl, K), "streams_per_gpu": K, "frame_ring": R,
                   "sharding": "stream s of the job on rank s mod N; no data-path collective; host-side gather of the result records",
                   "l2": "flushed between timed steps (256 MiB device write outside the timed events)",
                   "timing": "CUDA events on the launching stream around every tick, summed over the timed steps"},
        "e2e": {"value": n_frames / e2e_s, "unit": UNIT, "h2d_bytes_per_step": K * frame_bytes,
                "d2h_bytes_per_step": K * C.sizeof(binding.tt_result) + 4,
                "value_with_l2_flush": n_frames / e2e_flush_s,
                "serial_value": n_frames / e2e_serial_s,
                "timing": "host clock, pinned host frames, host->device copies and the device->host result read inside. value: three "
                          "submits in flight (tick i+2 submitted before tick i is synced), no cache flush (each step's input comes "
                          "from host memory); value_with_l2_flush: the same with a 256 MiB flush write in stream order between ticks, "
                          "its time included; serial_value: submit -> sync one tick at a time, flush outside the timed part"},
        "gpu_launches": launches1 - launches0,
        "roofline": roofline, "stages": stages, "clocks": clocks_main,
    }
    if latency is not None:
        line["latency"] = latency
    if staggered is not None:
        line["latency_staggered"] = staggered
    if sweep is not None:
        line["sweep"] = sweep
    if target is not None:
        line["target_config"] = target
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
    ap.add_argument("--ring", type=int, default=6, help="distinct frames per stream, reused cyclically")
    ap.add_argument("--paced-frames", type=int, default=600, help="frames per stream of the paced latency run (0: skip)")
    ap.add_argument("--staggered-frames", type=int, default=300,
                    help="frames per stream of the unsynchronised-arrival run through the batch planner (0: skip)")
    ap.add_argument("--window-ms", type=float, default=1.0, help="coalescing window of the batch planner")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", default="", help="comma-separated stream counts to measure in addition, e.g. 1,2,3,4,5,6,7,8")
    ap.add_argument("--sweep-steps", type=int, default=100)
    ap.add_argument("--sweep-paced-frames", type=int, default=200)
    ap.add_argument("--target-steps", type=int, default=10,
                    help="timed ticks of the scale-sweep configuration (cfg4, K=8) reported as target_config (0: skip)")
    ap.add_argument("--target-sweeps", type=int, default=1, help="also sweep the stream count at both sizes (0: skip)")
    ap.add_argument("--target-paced-frames", type=int, default=120, help="frames per stream of every sweep point's paced run")
    ap.add_argument("--study", default="", choices=["", "render", "hetero", "multi-model"],
                    help="run one of the latency studies instead of the benchmark line (1 GPU)")
    ap.add_argument("--study-frames", type=int, default=300, help="paced frames per stream and setting of a study")
    ap.add_argument("--study-streams", default="1,2,3,4,5,6", help="stream counts of the render study")
    ap.add_argument("--render-layers", type=int, default=8)
    ap.add_argument("--carve-sms", type=int, default=16, help="multiprocessors given to the carved-out render load")
    ap.add_argument("--hetero-k", type=int, default=3, help="streams per model in the heterogeneous study")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    if args.study == "render":
        return render_study(args)
    if args.study == "hetero":
        return hetero_study(args)
    if args.study == "multi-model":
        return multi_model_study(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
