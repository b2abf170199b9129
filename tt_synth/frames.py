"""Seeded uint8 RGB video frames standing in for the endoscopy video.

Two recipes (both HWC interleaved RGB, row pitch 3*W, top-left origin):

* "disc": uniform noise in [32, 96) plus one bright disc of radius 12 circling the image
  centre once every 8 frames (the tiny configuration).
* "endoscopy": smooth colour gradients that drift slowly in time, 1..7 rotating elliptical
  grey "tool" blobs on Lissajous paths, and integer noise in [-8, 8] per channel.

A frame is a pure function of (seed, frame index, shape), so streams can be generated in
any order and a ring of frames can be reproduced exactly.
"""
from __future__ import annotations

import math

import numpy as np

from .rng import raw_u64, uniform01

_TID_NOISE = 1000     # + frame index
_TID_BLOBS = 11


def _disc_frame(seed: int, t: int, w: int, h: int) -> np.ndarray:
    n = w * h * 3
    noise = (raw_u64(seed, _TID_NOISE + t, n) >> np.uint64(56)).astype(np.int64)  # 0..255
    img = (noise // 4 + 32).reshape(h, w, 3)
    cx = w / 2.0 + (w * 40.0 / 128.0) * math.cos(2.0 * math.pi * t / 8.0)
    cy = h / 2.0 + (h * 40.0 / 128.0) * math.sin(2.0 * math.pi * t / 8.0)
    r = 12.0 * min(w, h) / 128.0
    yy, xx = np.mgrid[0:h, 0:w]
    inside = (xx - cx) ** 2 + (yy - cy) ** 2 <= r * r
    img[inside] = np.array([240, 240, 230], dtype=np.int64)
    return img.astype(np.uint8)


def _endoscopy_frame(seed: int, t: int, w: int, h: int) -> np.ndarray:
    yy, xx = np.mgrid[0:h, 0:w].astype(np.float64)
    drift = math.sin(2.0 * math.pi * t / 240.0)
    r = 96.0 + 64.0 * xx / w + 10.0 * drift
    g = 56.0 + 48.0 * yy / h + 8.0 * math.sin(2.0 * math.pi * t / 310.0 + 1.0)
    b = 48.0 + 40.0 * (xx + yy) / (w + h) - 6.0 * drift
    img = np.stack([r, g, b], axis=-1)

    n_blobs = 1 + (seed % 7)
    p = uniform01(seed, _TID_BLOBS, n_blobs * 10).reshape(n_blobs, 10)
    for i in range(n_blobs):
        a = w / 20.0 + p[i, 0] * (w / 8.0 - w / 20.0)
        bb = h / 30.0 + p[i, 1] * (h / 10.0 - h / 30.0)
        fx, fy = 0.003 + 0.012 * p[i, 2], 0.004 + 0.011 * p[i, 3]
        phx, phy = 2.0 * math.pi * p[i, 4], 2.0 * math.pi * p[i, 5]
        cx = w * (0.5 + 0.38 * math.sin(2.0 * math.pi * fx * t + phx))
        cy = h * (0.5 + 0.38 * math.sin(2.0 * math.pi * fy * t + phy))
        theta = 2.0 * math.pi * (p[i, 6] + (0.002 + 0.006 * p[i, 7]) * t)
        grey = 200.0 + 40.0 * p[i, 8]
        ct, st = math.cos(theta), math.sin(theta)
        u = (xx - cx) * ct + (yy - cy) * st
        v = -(xx - cx) * st + (yy - cy) * ct
        inside = (u / a) ** 2 + (v / bb) ** 2 <= 1.0
        img[inside] = grey
    noise = (raw_u64(seed, _TID_NOISE + t, w * h * 3) % np.uint64(17)).astype(np.int64) - 8
    out = np.floor(img).astype(np.int64) + noise.reshape(h, w, 3)
    return np.clip(out, 0, 255).astype(np.uint8)


def make_frame(kind: str, seed: int, t: int, w: int, h: int) -> np.ndarray:
    """One uint8 [h][w][3] frame of the given recipe."""
    if kind == "disc":
        return _disc_frame(seed, t, w, h)
    if kind == "endoscopy":
        return _endoscopy_frame(seed, t, w, h)
    raise ValueError(f"unknown frame kind {kind!r}")


def make_frames(kind: str, seed: int, n_frames: int, w: int, h: int, start: int = 0) -> np.ndarray:
    """uint8 [n_frames][h][w][3], frame indices start..start+n_frames-1."""
    out = np.empty((n_frames, h, w, 3), dtype=np.uint8)
    for i in range(n_frames):
        out[i] = make_frame(kind, seed, start + i, w, h)
    return out
