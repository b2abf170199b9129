"""numpy-facing wrappers of the C oracle stages (argument marshalling only)."""
from __future__ import annotations

import ctypes as C
from typing import Optional, Tuple

import numpy as np

from .build import build

_lib = C.CDLL(build())

_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")
_u8p = np.ctypeslib.ndpointer(np.uint8, flags="C_CONTIGUOUS")
_i32p = np.ctypeslib.ndpointer(np.int32, flags="C_CONTIGUOUS")
_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")

_lib.ora_num_threads.restype = C.c_int
_lib.ora_set_threads.argtypes = [C.c_int]
_lib.ora_resize_axis.argtypes = [C.c_int, C.c_int, _i32p, _i32p, _f64p]
_lib.ora_preprocess.argtypes = [_u8p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double,
                                C.c_double, C.c_double, _f32p, _i32p, _i32p, _f64p, _i32p, _i32p, _f64p]
_lib.ora_conv_out.argtypes = [C.c_int, C.c_int]
_lib.ora_conv_out.restype = C.c_int
_lib.ora_conv3x3.argtypes = [_f32p, C.c_int, C.c_int, C.c_int, _f32p, C.c_void_p, C.c_int, C.c_int,
                             C.c_int, _f32p]
_lib.ora_convlstm_step.argtypes = [_f32p, C.c_int, _f32p, _f32p, C.c_int, C.c_int, C.c_int, _f32p,
                                   C.c_void_p, _f32p, _f32p, C.c_void_p]
_lib.ora_head.argtypes = [_f32p, C.c_int, C.c_int, C.c_int, _f32p, C.c_void_p, C.c_int, C.c_double,
                          _f32p, _f32p, _u8p]
_lib.ora_conf_mean_sigmoid.argtypes = [_f32p, C.c_int, C.c_int, C.c_int, _f32p]
_lib.ora_conf_gap_linear.argtypes = [_f32p, C.c_int, C.c_int, C.c_int, _f32p, C.c_void_p, C.c_int, _f32p]
_lib.ora_centroids.argtypes = [_u8p, C.c_int, C.c_int, C.c_int, _f32p, _f32p, _i32p]
_lib.ora_overlay.argtypes = [_u8p, C.c_int, C.c_int, C.c_int, _u8p, C.c_int, C.c_int, C.c_int, _u8p, _u8p]
_lib.ora_round_bf16.argtypes = [_f32p, C.c_size_t]


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _opt(a: Optional[np.ndarray]):
    if a is None:
        return None, None
    a = _f32(a)
    return a, a.ctypes.data_as(C.c_void_p)


def num_threads() -> int:
    return int(_lib.ora_num_threads())


def set_threads(n: int) -> None:
    _lib.ora_set_threads(int(n))


def resize_axis(n_in: int, n_out: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    i0 = np.empty(n_out, np.int32); i1 = np.empty(n_out, np.int32); fr = np.empty(n_out, np.float64)
    _lib.ora_resize_axis(n_in, n_out, i0, i1, fr)
    return i0, i1, fr


def preprocess(frame: np.ndarray, net_w: int, net_h: int, norm_div=255.0, norm_mean=0.5,
               norm_std=0.25, pitch: Optional[int] = None, src_w: Optional[int] = None):
    """frame uint8 [H][W][3] (or a flat pitched buffer with src_w given) -> fp32 [3][net_h][net_w]."""
    if frame.ndim == 3:
        src_h, src_w_, _ = frame.shape
        src_w = src_w_
        pitch = 3 * src_w if pitch is None else pitch
        buf = np.ascontiguousarray(frame, dtype=np.uint8).reshape(-1)
    else:
        buf = np.ascontiguousarray(frame, dtype=np.uint8).reshape(-1)
        src_h = buf.size // pitch
    dst = np.empty((3, net_h, net_w), np.float32)
    x0 = np.empty(net_w, np.int32); x1 = np.empty(net_w, np.int32); fx = np.empty(net_w, np.float64)
    y0 = np.empty(net_h, np.int32); y1 = np.empty(net_h, np.int32); fy = np.empty(net_h, np.float64)
    _lib.ora_preprocess(buf, src_w, src_h, pitch, net_w, net_h, norm_div, norm_mean, norm_std, dst,
                        x0, x1, fx, y0, y1, fy)
    return dst


def conv3x3(x: np.ndarray, w: np.ndarray, b: Optional[np.ndarray], stride: int = 1, relu: bool = False):
    """x [Cin][H][W], w [Cout][Cin][3][3], b [Cout] or None -> [Cout][Ho][Wo]."""
    x = _f32(x); w = _f32(w)
    cin, h, wd = x.shape
    cout = w.shape[0]
    assert w.shape == (cout, cin, 3, 3)
    ho, wo = _lib.ora_conv_out(h, stride), _lib.ora_conv_out(wd, stride)
    out = np.empty((cout, ho, wo), np.float32)
    bk, bp = _opt(b)
    _lib.ora_conv3x3(x, cin, h, wd, w, bp, cout, stride, int(relu), out)
    return out


def convlstm_step(x, h, c, w, b, return_gates: bool = False):
    """x [Cx][H][W], h,c [Ch][H][W], w [4Ch][Cx+Ch][3][3], b [4Ch] -> (h', c'[, gates])."""
    x = _f32(x); h = _f32(h); c = _f32(c); w = _f32(w)
    cx, hm, wm = x.shape
    ch = h.shape[0]
    assert w.shape == (4 * ch, cx + ch, 3, 3) and c.shape == h.shape == (ch, hm, wm)
    h2 = np.empty_like(h); c2 = np.empty_like(c)
    gates = np.empty((4 * ch, hm, wm), np.float32) if return_gates else None
    bk, bp = _opt(b)
    gp = gates.ctypes.data_as(C.c_void_p) if gates is not None else None
    _lib.ora_convlstm_step(x, cx, h, c, ch, hm, wm, w, bp, h2, c2, gp)
    return (h2, c2, gates) if return_gates else (h2, c2)


def head(h, w, b, thr: float = 0.5):
    """h [Ch][H][W], w [T][Ch] -> (z, p, mask) each [T][H][W]."""
    h = _f32(h); w = _f32(w)
    ch, hm, wm = h.shape
    T = w.shape[0]
    z = np.empty((T, hm, wm), np.float32); p = np.empty_like(z); m = np.empty((T, hm, wm), np.uint8)
    bk, bp = _opt(b)
    _lib.ora_head(h, ch, hm, wm, w, bp, T, thr, z, p, m)
    return z, p, m


def conf_mean_sigmoid(p):
    p = _f32(p); T, hm, wm = p.shape
    conf = np.empty(T, np.float32)
    _lib.ora_conf_mean_sigmoid(p, T, hm, wm, conf)
    return conf


def conf_gap_linear(h, w, b):
    h = _f32(h); w = _f32(w); ch, hm, wm = h.shape; T = w.shape[0]
    conf = np.empty(T, np.float32)
    bk, bp = _opt(b)
    _lib.ora_conf_gap_linear(h, ch, hm, wm, w, bp, T, conf)
    return conf


def centroids(mask):
    mask = np.ascontiguousarray(mask, dtype=np.uint8); T, hm, wm = mask.shape
    cx = np.empty(T, np.float32); cy = np.empty(T, np.float32); n = np.empty(T, np.int32)
    _lib.ora_centroids(mask, T, hm, wm, cx, cy, n)
    return cx, cy, n


def overlay(frame, mask, palette):
    frame = np.ascontiguousarray(frame, dtype=np.uint8); sh, sw, _ = frame.shape
    mask = np.ascontiguousarray(mask, dtype=np.uint8); T, hm, wm = mask.shape
    pal = np.ascontiguousarray(np.asarray(palette, dtype=np.uint8)[:T]).reshape(-1)
    dst = np.empty((sh, sw, 4), np.uint8)
    _lib.ora_overlay(frame.reshape(-1), sw, sh, 3 * sw, mask, T, hm, wm, pal, dst)
    return dst


def render_layers(frame, mask, palette, layers: int):
    """Multi-layer stand-in for the visualisation load: the S6 blend applied `layers` times in sequence, layer l
    with the palette rotated by l (tool t takes colour (t + l) mod T), each layer on the previous layer's RGB."""
    if layers < 1:
        raise ValueError("layers >= 1 required")
    T = np.asarray(mask).shape[0]
    pal = [tuple(int(v) for v in c) for c in np.asarray(palette, dtype=np.uint8)[:T]]
    rgb = np.ascontiguousarray(frame, dtype=np.uint8)
    out = None
    for l in range(layers):
        out = overlay(rgb, mask, [pal[(t + l) % T] for t in range(T)])
        rgb = np.ascontiguousarray(out[..., :3])
    return out


def round_bf16(a):
    out = np.array(a, dtype=np.float32, order="C", copy=True)
    _lib.ora_round_bf16(out.reshape(-1), out.size)
    return out
