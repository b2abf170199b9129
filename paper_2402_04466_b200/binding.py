"""ctypes binding of libtt.so: same names as the C ABI in include/tt.h, argument marshalling only.

torch is used for device memory and streams; every step of the path runs in the library's
kernels.  If the library cannot be loaded (and cannot be built with nvcc) calls raise:
there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

TT_ABI_VERSION = 1
TT_MAX_STREAMS = 8
TT_MAX_IN_FLIGHT = 3
TT_MAX_TOOLS = 8
TT_MAX_ENC = 4

TT_OK = 0
STATUS_NAMES = {0: "TT_OK", 1: "TT_ERR_INVALID_ARG", 2: "TT_ERR_UNSUPPORTED", 3: "TT_ERR_OOM", 4: "TT_ERR_CUDA",
                5: "TT_ERR_ADMISSION", 6: "TT_ERR_NOT_READY", 7: "TT_ERR_TIMEOUT", 8: "TT_ERR_DEVICE_STATUS"}
TT_FP32, TT_BF16 = 0, 1
TT_OPT_PLAIN_LAUNCHES, TT_OPT_FEED_FORWARD, TT_OPT_CTA_PAIRS, TT_OPT_NO_POST_TC, TT_OPT_RESERVED_SMS = 0, 1, 2, 3, 4
TT_OPT_ENC_ONE_PER_SM, TT_OPT_NO_HALO, TT_OPT_FUSED_PRE = 5, 6, 7
TT_CONF_MEAN_SIGMOID, TT_CONF_GAP_LINEAR = 0, 1
TENSOR_IDS = {"pre": 0, "enc0": 1, "enc1": 2, "enc2": 3, "enc3": 4, "h": 8, "c": 9, "logits": 10, "prob": 11}

EXPORTED_SYMBOLS = [
    "tt_abi_version", "tt_create", "tt_destroy", "tt_last_error", "tt_map_size", "tt_state_create",
    "tt_state_reset", "tt_state_export", "tt_state_import", "tt_submit_frames", "tt_sync", "tt_debug_tensor",
    "tt_set_profiling", "tt_get_stage_times", "tt_get_counters", "tt_query", "tt_debug_expire_wait",
    "tt_sched_create", "tt_sched_destroy", "tt_sched_admit", "tt_sched_release", "tt_sched_arrive", "tt_sched_next",
    "tt_sched_complete", "tt_sched_predict_ms", "tt_sched_stats",
    "tt_preprocess", "tt_postprocess_scratch_bytes", "tt_postprocess", "tt_postprocess_static", "tt_overlay", "tt_render_layers",
]
TT_POSTPROCESS_STATIC_SCRATCH_BYTES = 32 << 10
STAGE_NAMES = ["h2d", "preprocess", "enc0", "enc1", "enc2", "enc3", "convlstm", "postprocess", "overlay"]


class TTError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class tt_config(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("abi_version", C.c_uint32),
        ("device", C.c_int32), ("max_streams", C.c_int32),
        ("src_w", C.c_int32), ("src_h", C.c_int32), ("src_pitch", C.c_int32),
        ("net_w", C.c_int32), ("net_h", C.c_int32),
        ("norm_div", C.c_float), ("norm_mean", C.c_float), ("norm_std", C.c_float),
        ("n_enc", C.c_int32), ("enc_cout", C.c_int32 * TT_MAX_ENC), ("enc_stride", C.c_int32 * TT_MAX_ENC),
        ("hidden", C.c_int32), ("n_tools", C.c_int32), ("precision", C.c_int32), ("conf_mode", C.c_int32),
        ("threshold", C.c_float), ("overlay", C.c_int32),
        ("palette", (C.c_uint8 * 3) * TT_MAX_TOOLS), ("options", C.c_uint8 * 8),
        ("cuda_stream", C.c_void_p), ("sync_timeout_ns", C.c_uint64),
    ]


class tt_weights(C.Structure):
    _fields_ = [
        ("enc_w", C.c_void_p * TT_MAX_ENC), ("enc_b", C.c_void_p * TT_MAX_ENC),
        ("lstm_w", C.c_void_p), ("lstm_b", C.c_void_p), ("head_w", C.c_void_p), ("head_b", C.c_void_p),
        ("conf_w", C.c_void_p), ("conf_b", C.c_void_p),
    ]


class tt_frame(C.Structure):
    _fields_ = [("data", C.c_void_p), ("on_device", C.c_int32), ("reserved_", C.c_int32),
                ("frame_index", C.c_uint64), ("arrival_ns", C.c_uint64)]


class tt_result(C.Structure):
    _fields_ = [("frame_index", C.c_uint64), ("arrival_ns", C.c_uint64),
                ("conf", C.c_float * TT_MAX_TOOLS), ("cx", C.c_float * TT_MAX_TOOLS), ("cy", C.c_float * TT_MAX_TOOLS),
                ("count", C.c_int32 * TT_MAX_TOOLS),
                ("masks_dev", C.c_void_p), ("probs_dev", C.c_void_p), ("overlay_dev", C.c_void_p),
                ("gpu_ms", C.c_float), ("reserved_", C.c_int32)]


class tt_sched_config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("max_streams", C.c_int32), ("max_in_flight", C.c_int32),
                ("budget_fraction", C.c_float), ("window_ns", C.c_uint64), ("deadline_ns", C.c_uint64),
                ("tick_ms_base", C.c_float), ("tick_ms_per_stream", C.c_float)]


_LIB = None
LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libtt.so")


def load_library(build_if_missing: bool = True) -> C.CDLL:
    """dlopen libtt.so (building it in-tree with nvcc when absent or stale) and declare prototypes."""
    global _LIB
    if _LIB is not None:
        return _LIB
    if build_if_missing:
        from .build import build
        build()
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2402_04466_b200.build`; "
                           "there is no CPU fallback")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    lib.tt_abi_version.restype = C.c_uint32
    lib.tt_create.argtypes = [C.POINTER(tt_config), C.POINTER(tt_weights), C.POINTER(vp)]
    lib.tt_destroy.argtypes = [vp]
    lib.tt_last_error.argtypes = [vp]
    lib.tt_last_error.restype = C.c_char_p
    lib.tt_map_size.argtypes = [vp, C.POINTER(i32), C.POINTER(i32)]
    lib.tt_state_create.argtypes = [vp, C.POINTER(vp)]
    lib.tt_state_reset.argtypes = [vp, vp]
    lib.tt_state_export.argtypes = [vp, vp, vp, vp]
    lib.tt_state_import.argtypes = [vp, vp, vp, vp]
    lib.tt_submit_frames.argtypes = [vp, i32, C.POINTER(tt_frame), C.POINTER(vp)]
    lib.tt_sync.argtypes = [vp, C.POINTER(tt_result)]
    lib.tt_debug_tensor.argtypes = [vp, vp, i32, vp, C.c_size_t]
    lib.tt_set_profiling.argtypes = [vp, i32]
    lib.tt_get_stage_times.argtypes = [vp, C.POINTER(C.c_float)]
    lib.tt_get_counters.argtypes = [vp, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    lib.tt_query.argtypes = [vp]
    lib.tt_debug_expire_wait.argtypes = [vp, C.c_uint64]
    u64p = C.POINTER(C.c_uint64)
    lib.tt_sched_create.argtypes = [C.POINTER(tt_sched_config), C.POINTER(vp)]
    lib.tt_sched_destroy.argtypes = [vp]
    lib.tt_sched_admit.argtypes = [vp, C.POINTER(i32)]
    lib.tt_sched_release.argtypes = [vp, i32]
    lib.tt_sched_arrive.argtypes = [vp, i32, C.c_uint64, C.c_uint64]
    lib.tt_sched_next.argtypes = [vp, C.c_uint64, C.POINTER(i32), C.POINTER(i32), u64p, u64p, u64p]
    lib.tt_sched_complete.argtypes = [vp, f32, C.c_uint64]
    lib.tt_sched_predict_ms.argtypes = [vp, i32, C.POINTER(f32)]
    lib.tt_sched_stats.argtypes = [vp, u64p, u64p, u64p, u64p]
    lib.tt_preprocess.argtypes = [vp, i32, i64, i32, i32, i32, vp, i32, i32, f32, f32, f32, vp]
    lib.tt_postprocess_scratch_bytes.argtypes = [i32, i32, i32, i32, i32]
    lib.tt_postprocess_scratch_bytes.restype = C.c_size_t
    lib.tt_postprocess.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, i32, f32, vp, vp, vp, vp, vp, vp]
    lib.tt_postprocess_static.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, i32, f32, vp, vp, vp, vp, vp]
    lib.tt_overlay.argtypes = [vp, i32, i64, i32, i32, i32, vp, i32, i32, i32, vp, vp, vp]
    lib.tt_render_layers.argtypes = [vp, i32, i64, i32, i32, i32, vp, i32, i32, i32, vp, i32, i32, vp, vp]
    for name in EXPORTED_SYMBOLS:
        getattr(lib, name)  # AttributeError here means the library does not export what tt.h declares
    _LIB = lib
    return lib


def _check(lib, status: int, ctx=None):
    if status != TT_OK:
        msg = lib.tt_last_error(ctx)
        raise TTError(status, msg.decode() if msg else "")


def make_config(wl, max_streams: int = 1, device: int = 0, overlay: Optional[bool] = None,
                cuda_stream: int = 0, sync_timeout_ns: int = 0, precision: Optional[str] = None,
                plain_launches: bool = False, cta_pairs: bool = False, post_tc: bool = True,
                reserved_sms: int = 0, enc_two_per_sm: bool = True, halo: bool = True,
                fused_pre: bool = False) -> tt_config:
    """Fill a tt_config from any object carrying the workload attributes (src_w, net_w, enc_cout, ...).

    plain_launches=True makes every tick launch its kernels one by one instead of replaying a CUDA graph.
    fused_pre=True runs the preprocessing inside the first encoder layer (bf16 path; same bits, measured slower)."""
    cfg = tt_config()
    cfg.struct_size = C.sizeof(tt_config)
    cfg.abi_version = TT_ABI_VERSION
    cfg.device = device
    cfg.max_streams = max_streams
    cfg.src_w, cfg.src_h, cfg.src_pitch = wl.src_w, wl.src_h, getattr(wl, "src_pitch", 3 * wl.src_w)
    cfg.net_w, cfg.net_h = wl.net_w, wl.net_h
    cfg.norm_div, cfg.norm_mean, cfg.norm_std = wl.norm_div, wl.norm_mean, wl.norm_std
    cfg.n_enc = len(wl.enc_cout)
    for i, (co, s) in enumerate(zip(wl.enc_cout, wl.enc_stride)):
        cfg.enc_cout[i] = co
        cfg.enc_stride[i] = s
    cfg.hidden, cfg.n_tools = wl.hidden, wl.n_tools
    prec = precision or wl.precision
    cfg.precision = TT_BF16 if prec == "bf16" else TT_FP32
    cfg.conf_mode = TT_CONF_GAP_LINEAR if wl.conf_mode == "gap_linear" else TT_CONF_MEAN_SIGMOID
    cfg.threshold = wl.threshold
    cfg.overlay = int(wl.overlay if overlay is None else overlay)
    for t in range(TT_MAX_TOOLS):
        for k in range(3):
            cfg.palette[t][k] = wl.palette[t][k]
    cfg.cuda_stream = cuda_stream or None
    cfg.sync_timeout_ns = sync_timeout_ns
    cfg.options[TT_OPT_PLAIN_LAUNCHES] = 1 if plain_launches else 0
    cfg.options[TT_OPT_FEED_FORWARD] = 0 if getattr(wl, "recurrent", True) else 1
    cfg.options[TT_OPT_CTA_PAIRS] = 1 if cta_pairs else 0
    cfg.options[TT_OPT_NO_POST_TC] = 0 if post_tc else 1
    cfg.options[TT_OPT_RESERVED_SMS] = reserved_sms
    cfg.options[TT_OPT_ENC_ONE_PER_SM] = 0 if enc_two_per_sm else 1
    cfg.options[TT_OPT_NO_HALO] = 0 if halo else 1
    cfg.options[TT_OPT_FUSED_PRE] = 1 if fused_pre else 0
    return cfg


def _result_to_dict(r: tt_result, n_tools: int) -> Dict:
    return {
        "frame_index": int(r.frame_index), "arrival_ns": int(r.arrival_ns),
        "conf": np.array(r.conf[:n_tools], np.float32), "cx": np.array(r.cx[:n_tools], np.float32),
        "cy": np.array(r.cy[:n_tools], np.float32), "count": np.array(r.count[:n_tools], np.int32),
        "masks_dev": r.masks_dev, "probs_dev": r.probs_dev, "overlay_dev": r.overlay_dev, "gpu_ms": float(r.gpu_ms),
    }


class Context:
    """tt_create .. tt_destroy with the same call names as the C ABI."""

    def __init__(self, cfg: tt_config, weights: Dict[str, np.ndarray]):
        self.lib = load_library()
        self.cfg = cfg
        self._keep = []
        w = tt_weights()

        def ptr(a):
            a = np.ascontiguousarray(a, dtype=np.float32)
            self._keep.append(a)
            return a.ctypes.data_as(C.c_void_p)

        for l in range(cfg.n_enc):
            w.enc_w[l] = ptr(weights[f"enc_w{l}"]).value
            w.enc_b[l] = ptr(weights[f"enc_b{l}"]).value
        if "lstm_w" in weights:
            w.lstm_w, w.lstm_b = ptr(weights["lstm_w"]), ptr(weights["lstm_b"])
        w.head_w, w.head_b = ptr(weights["head_w"]), ptr(weights["head_b"])
        if "conf_w" in weights:
            w.conf_w, w.conf_b = ptr(weights["conf_w"]), ptr(weights["conf_b"])
        h = C.c_void_p()
        st = self.lib.tt_create(C.byref(cfg), C.byref(w), C.byref(h))
        _check(self.lib, st, None)
        self.handle = h
        self._keep.clear()
        hm, wm = C.c_int32(), C.c_int32()
        _check(self.lib, self.lib.tt_map_size(self.handle, C.byref(hm), C.byref(wm)), self.handle)
        self.hm, self.wm = hm.value, wm.value
        self.n_tools, self.hidden = cfg.n_tools, cfg.hidden
        self._ks = []                # stream counts of the submits in flight, oldest first
        self._inflight_keep = []     # keeps the frame tensors of in-flight submits alive

    # -- lifetime
    def destroy(self):
        if getattr(self, "handle", None):
            self.lib.tt_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- states
    def state_create(self) -> C.c_void_p:
        s = C.c_void_p()
        _check(self.lib, self.lib.tt_state_create(self.handle, C.byref(s)), self.handle)
        return s

    def state_reset(self, st):
        _check(self.lib, self.lib.tt_state_reset(self.handle, st), self.handle)

    def state_export(self, st):
        shape = (self.hidden, self.hm, self.wm)
        h = np.empty(shape, np.float32)
        c = np.empty(shape, np.float32)
        _check(self.lib, self.lib.tt_state_export(self.handle, st, h.ctypes.data, c.ctypes.data), self.handle)
        return h, c

    def state_import(self, st, h, c):
        h = np.ascontiguousarray(h, np.float32)
        c = np.ascontiguousarray(c, np.float32)
        _check(self.lib, self.lib.tt_state_import(self.handle, st, h.ctypes.data, c.ctypes.data), self.handle)

    # -- per tick
    def submit_frames(self, frames: Sequence, states: Sequence, frame_index: int = 0,
                      arrival_ns: Optional[Sequence[int]] = None):
        """frames: torch uint8 tensors, CUDA (device-resident) or pinned CPU; one per stream."""
        K = len(frames)
        fr = (tt_frame * max(K, 1))()
        for k, f in enumerate(frames):
            fr[k].data = f.data_ptr()
            fr[k].on_device = 1 if f.is_cuda else 0
            fr[k].frame_index = frame_index
            fr[k].arrival_ns = int(arrival_ns[k]) if arrival_ns is not None else 0
        sts = (C.c_void_p * max(K, 1))(*[s.value if isinstance(s, C.c_void_p) else s for s in states])
        st = self.lib.tt_submit_frames(self.handle, K, fr, sts)
        _check(self.lib, st, self.handle)
        self._ks.append(K)
        self._inflight_keep.append(list(frames))

    def submit_raw(self, K: int, frame_array, state_array) -> int:
        """Pre-marshalled arrays (tt_frame[K], void*[K]); returns the status without raising."""
        st = self.lib.tt_submit_frames(self.handle, K, frame_array, state_array)
        if st == TT_OK:
            self._ks.append(K)
            self._inflight_keep.append(None)
        return st

    def sync(self) -> List[Dict]:
        res = (tt_result * TT_MAX_STREAMS)()
        st = self.lib.tt_sync(self.handle, res)
        if st == 8 and self._ks:                 # TT_ERR_DEVICE_STATUS: the submit is over, its results are invalid
            self._ks.pop(0)
            self._inflight_keep.pop(0)
        _check(self.lib, st, self.handle)        # any other error (a timeout, say) leaves the submit in flight
        k_done = self._ks.pop(0)                 # submits complete oldest first
        self._inflight_keep.pop(0)
        return [_result_to_dict(res[k], self.n_tools) for k in range(k_done)]

    def sync_raw(self, result_array) -> int:
        st = self.lib.tt_sync(self.handle, result_array)
        if st in (TT_OK, 8) and self._ks:
            self._ks.pop(0)
            self._inflight_keep.pop(0)
        return st

    def set_profiling(self, on: bool):
        _check(self.lib, self.lib.tt_set_profiling(self.handle, int(on)), self.handle)

    def get_stage_times(self) -> Dict[str, float]:
        ms = (C.c_float * len(STAGE_NAMES))()
        _check(self.lib, self.lib.tt_get_stage_times(self.handle, ms), self.handle)
        return {n: float(ms[i]) for i, n in enumerate(STAGE_NAMES) if ms[i] >= 0}

    def get_counters(self):
        a, b = C.c_uint64(), C.c_uint64()
        _check(self.lib, self.lib.tt_get_counters(self.handle, C.byref(a), C.byref(b)), self.handle)
        return int(a.value), int(b.value)

    def query(self) -> bool:
        """True when the oldest submit in flight has finished (tt_sync would not block)."""
        return self.lib.tt_query(self.handle) == TT_OK

    def debug_expire_wait(self, limit_cycles: int):
        """Enqueue the failure-path probe: a bounded device-side wait that runs out after limit_cycles."""
        _check(self.lib, self.lib.tt_debug_expire_wait(self.handle, limit_cycles), self.handle)

    def last_error(self) -> str:
        m = self.lib.tt_last_error(self.handle)
        return m.decode() if m else ""

    def debug_tensor(self, st, which: str) -> np.ndarray:
        if which == "pre":
            shape = (3, self.cfg.net_h, self.cfg.net_w)
        elif which.startswith("enc"):
            l = int(which[3:])
            h, w = self.cfg.net_h, self.cfg.net_w
            for i in range(l + 1):
                s = self.cfg.enc_stride[i]
                h, w = (h + 2 - 3) // s + 1, (w + 2 - 3) // s + 1
            shape = (self.cfg.enc_cout[l], h, w)
        elif which in ("h", "c"):
            shape = (self.hidden, self.hm, self.wm)
        else:
            shape = (self.n_tools, self.hm, self.wm)
        out = np.empty(shape, np.float32)
        _check(self.lib, self.lib.tt_debug_tensor(self.handle, st, TENSOR_IDS[which], out.ctypes.data, out.size), self.handle)
        return out

    # -- device views of the last results (torch, zero-copy is not needed for tests: copy out)
    def fetch_masks(self, result: Dict) -> np.ndarray:
        return _copy_from_device(result["masks_dev"], (self.n_tools, self.hm, self.wm), np.uint8)

    def fetch_probs(self, result: Dict) -> np.ndarray:
        return _copy_from_device(result["probs_dev"], (self.n_tools, self.hm, self.wm), np.float32)

    def fetch_overlay(self, result: Dict) -> np.ndarray:
        return _copy_from_device(result["overlay_dev"], (self.cfg.src_h, self.cfg.src_w, 4), np.uint8)


class Scheduler:
    """tt_sched_*: batch planner for unsynchronised arrivals (host logic only, usable without a GPU)."""

    NEVER = 2 ** 64 - 1

    def __init__(self, max_streams: int, window_ns: int, deadline_ns: int = 16_666_667, max_in_flight: int = 2,
                 budget_fraction: float = 0.5, tick_ms_base: float = 0.1, tick_ms_per_stream: float = 0.02):
        self.lib = load_library()
        cfg = tt_sched_config(C.sizeof(tt_sched_config), max_streams, max_in_flight, budget_fraction, window_ns,
                              deadline_ns, tick_ms_base, tick_ms_per_stream)
        h = C.c_void_p()
        st = self.lib.tt_sched_create(C.byref(cfg), C.byref(h))
        if st != TT_OK:
            raise TTError(st, "tt_sched_create")
        self.handle, self.max_streams = h, max_streams

    def destroy(self):
        if self.handle:
            self.lib.tt_sched_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def admit(self) -> int:
        sid = C.c_int32()
        st = self.lib.tt_sched_admit(self.handle, C.byref(sid))
        if st != TT_OK:
            raise TTError(st, "stream refused by admission control")
        return sid.value

    def release(self, stream_id: int):
        st = self.lib.tt_sched_release(self.handle, stream_id)
        if st != TT_OK:
            raise TTError(st, "tt_sched_release")

    def arrive(self, stream_id: int, frame_index: int, t_ns: int) -> bool:
        """False when the frame was dropped because the stream's previous frame is still waiting."""
        st = self.lib.tt_sched_arrive(self.handle, stream_id, frame_index, t_ns)
        if st == TT_OK:
            return True
        if st == 5:
            return False
        raise TTError(st, "tt_sched_arrive")

    def next(self, now_ns: int):
        """-> (batch, wake_ns); batch is a list of (stream_id, frame_index, arrival_ns), empty when nothing launches now."""
        K = C.c_int32()
        ids = (C.c_int32 * TT_MAX_STREAMS)()
        fi = (C.c_uint64 * TT_MAX_STREAMS)()
        ar = (C.c_uint64 * TT_MAX_STREAMS)()
        wake = C.c_uint64()
        st = self.lib.tt_sched_next(self.handle, now_ns, C.byref(K), ids, fi, ar, C.byref(wake))
        if st != TT_OK:
            raise TTError(st, "tt_sched_next")
        return [(ids[i], fi[i], ar[i]) for i in range(K.value)], wake.value

    def complete(self, gpu_ms: float, done_ns: int):
        st = self.lib.tt_sched_complete(self.handle, gpu_ms, done_ns)
        if st != TT_OK:
            raise TTError(st, "tt_sched_complete")

    def predict_ms(self, K: int) -> float:
        ms = C.c_float()
        st = self.lib.tt_sched_predict_ms(self.handle, K, C.byref(ms))
        if st != TT_OK:
            raise TTError(st, "tt_sched_predict_ms")
        return ms.value

    def stats(self):
        a, b, c, d = C.c_uint64(), C.c_uint64(), C.c_uint64(), C.c_uint64()
        self.lib.tt_sched_stats(self.handle, C.byref(a), C.byref(b), C.byref(c), C.byref(d))
        return {"batches": a.value, "frames": b.value, "dropped": c.value, "deadline_misses": d.value}


class _DeviceView:
    """Exposes a raw device pointer through __cuda_array_interface__ so torch can wrap it."""

    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (int(ptr), False),
                                         "version": 2, "strides": None}


def device_tensor(ptr: int, shape, dtype):
    """torch tensor aliasing library-owned device memory (valid until the next submit)."""
    import torch
    typestr = {np.uint8: "|u1", np.float32: "<f4", np.int32: "<i4"}[dtype]
    return torch.as_tensor(_DeviceView(ptr, shape, typestr), device="cuda")


def _copy_from_device(ptr: int, shape, dtype) -> np.ndarray:
    return device_tensor(ptr, shape, dtype).cpu().numpy().copy()


# ------------------------------------------------------------------------ stage-level calls
def _stream_ptr(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


def preprocess(src, src_w: int, src_h: int, src_pitch: int, net_w: int, net_h: int, norm_div=255.0, norm_mean=0.5,
               norm_std=0.25, stream=None):
    """src: torch uint8 CUDA tensor [K][src_h*src_pitch] -> torch fp32 [K][3][net_h][net_w]."""
    import torch
    lib = load_library()
    K = src.shape[0]
    dst = torch.empty((K, 3, net_h, net_w), dtype=torch.float32, device=src.device)
    st = lib.tt_preprocess(src.data_ptr(), K, src.stride(0), src_w, src_h, src_pitch, dst.data_ptr(), net_w, net_h,
                           norm_div, norm_mean, norm_std, _stream_ptr(stream))
    _check(lib, st, None)
    return dst


def postprocess(h, channels_last: bool, head_w, head_b, conf_w=None, conf_b=None, conf_mode="mean_sigmoid",
                threshold=0.5, stream=None):
    """h: torch fp32 CUDA [K][Hm][Wm][Ch] (channels_last) or [K][Ch][Hm][Wm]; returns dict of outputs."""
    import torch
    lib = load_library()
    if channels_last:
        K, hm, wm, ch = h.shape
    else:
        K, ch, hm, wm = h.shape
    T = head_w.shape[0]
    dev = h.device
    logits = torch.empty((K, T, hm, wm), dtype=torch.float32, device=dev)
    probs = torch.empty_like(logits)
    masks = torch.empty((K, T, hm, wm), dtype=torch.uint8, device=dev)
    results = torch.zeros((K, C.sizeof(tt_result)), dtype=torch.uint8, device=dev)
    scratch = torch.empty((max(int(lib.tt_postprocess_scratch_bytes(K, hm, wm, ch, T)), 256),), dtype=torch.uint8, device=dev)
    mode = TT_CONF_GAP_LINEAR if conf_mode == "gap_linear" else TT_CONF_MEAN_SIGMOID
    st = lib.tt_postprocess(h.data_ptr(), int(channels_last), K, hm, wm, ch, T, head_w.data_ptr(), head_b.data_ptr(),
                            conf_w.data_ptr() if conf_w is not None else None,
                            conf_b.data_ptr() if conf_b is not None else None, mode, threshold, logits.data_ptr(),
                            probs.data_ptr(), masks.data_ptr(), results.data_ptr(), scratch.data_ptr(), _stream_ptr(stream))
    _check(lib, st, None)
    torch.cuda.synchronize()
    raw = results.cpu().numpy().tobytes()
    recs = [_result_to_dict(tt_result.from_buffer_copy(raw[k * C.sizeof(tt_result):(k + 1) * C.sizeof(tt_result)]), T)
            for k in range(K)]
    return {"logits": logits, "probs": probs, "masks": masks, "results": recs}


def postprocess_static(h, channels_last: bool, head_w, head_b, conf_w=None, conf_b=None, conf_mode="mean_sigmoid",
                       threshold=0.5, stream=None, out=None):
    """tt_postprocess_static: like postprocess(), but the library call itself allocates nothing.

    For callers that cannot allocate device memory while they run (a frame loop with a fixed
    memory budget, a plug-in fed by its host's allocator).  The output tensors are the caller's:
    pass them as `out` (dict with logits, probs, masks, results) to reuse buffers across calls;
    when `out` is None this helper creates them with torch before calling into the library.
    """
    import torch
    lib = load_library()
    if channels_last:
        K, hm, wm, ch = h.shape
    else:
        K, ch, hm, wm = h.shape
    T = head_w.shape[0]
    dev = h.device
    if out is None:
        out = {"logits": torch.empty((K, T, hm, wm), dtype=torch.float32, device=dev),
               "probs": torch.empty((K, T, hm, wm), dtype=torch.float32, device=dev),
               "masks": torch.empty((K, T, hm, wm), dtype=torch.uint8, device=dev),
               "results_raw": torch.zeros((K, C.sizeof(tt_result)), dtype=torch.uint8, device=dev)}
    mode = TT_CONF_GAP_LINEAR if conf_mode == "gap_linear" else TT_CONF_MEAN_SIGMOID
    st = lib.tt_postprocess_static(h.data_ptr(), int(channels_last), K, hm, wm, ch, T, head_w.data_ptr(), head_b.data_ptr(),
                                   conf_w.data_ptr() if conf_w is not None else None,
                                   conf_b.data_ptr() if conf_b is not None else None, mode, threshold,
                                   out["logits"].data_ptr(), out["probs"].data_ptr(), out["masks"].data_ptr(),
                                   out["results_raw"].data_ptr(), _stream_ptr(stream))
    _check(lib, st, None)
    torch.cuda.synchronize()
    raw = out["results_raw"].cpu().numpy().tobytes()
    n = C.sizeof(tt_result)
    out["results"] = [_result_to_dict(tt_result.from_buffer_copy(raw[k * n:(k + 1) * n]), T) for k in range(K)]
    return out


def overlay(src, src_w: int, src_h: int, src_pitch: int, masks, palette, stream=None):
    """src: torch uint8 CUDA [K][src_h*src_pitch]; masks uint8 CUDA [K][T][Hm][Wm] -> uint8 [K][src_h][src_w][4]."""
    import torch
    lib = load_library()
    K, T, hm, wm = masks.shape
    pal = np.ascontiguousarray(np.asarray(palette, np.uint8)[:T]).reshape(-1)
    dst = torch.empty((K, src_h, src_w, 4), dtype=torch.uint8, device=src.device)
    st = lib.tt_overlay(src.data_ptr(), K, src.stride(0), src_w, src_h, src_pitch, masks.data_ptr(), T, hm, wm,
                        pal.ctypes.data, dst.data_ptr(), _stream_ptr(stream))
    _check(lib, st, None)
    return dst


def render_layers(src, src_w: int, src_h: int, src_pitch: int, masks, palette, layers: int, carve_ctas: int = 0, stream=None,
                  out=None):
    """tt_render_layers: src uint8 CUDA [K][src_h*src_pitch], masks uint8 CUDA [K][T][Hm][Wm] -> uint8 [K][src_h][src_w][4]."""
    import torch
    lib = load_library()
    K, T, hm, wm = masks.shape
    pal = np.ascontiguousarray(np.asarray(palette, np.uint8)[:T]).reshape(-1)
    dst = out if out is not None else torch.empty((K, src_h, src_w, 4), dtype=torch.uint8, device=src.device)
    st = lib.tt_render_layers(src.data_ptr(), K, src.stride(0), src_w, src_h, src_pitch, masks.data_ptr(), T, hm, wm,
                              pal.ctypes.data, layers, carve_ctas, dst.data_ptr(), _stream_ptr(stream))
    _check(lib, st, None)
    return dst
