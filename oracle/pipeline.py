"""Per-frame chain of the oracle stages with recurrent state (test infrastructure only).

Order follows the operator chain of the paper's Endoscopy Tool Tracking application
(Section III-A): format conversion (resize + normalise), recurrent inference (conv encoder
then one ConvLSTM cell step), tool-tracking post-processing (mask head, threshold,
confidence, centroid), and the overlay that stands in for the visualisation operator.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np

from . import stages as S


@dataclass
class FrameOutput:
    pre: np.ndarray
    enc: List[np.ndarray]
    h: np.ndarray
    c: np.ndarray
    z: np.ndarray
    p: np.ndarray
    mask: np.ndarray
    conf: np.ndarray
    cx: np.ndarray
    cy: np.ndarray
    count: np.ndarray
    overlay: Optional[np.ndarray]


class OraclePipeline:
    """One stream: weights + (h, c).  `wl` is any object with the Workload attributes.

    mirror_bf16=True rounds to bf16 exactly those activations that a bf16 tensor-core path
    must round before a contraction (the network input of the first layer, every encoder
    output and the copy of h fed back into the ConvLSTM convolution); state, heads and everything observable stay fp32.
    """

    def __init__(self, wl, weights: Dict[str, np.ndarray], mirror_bf16: bool = False):
        self.wl = wl
        self.w = weights
        self.mirror = bool(mirror_bf16)
        hm, wm = wl.map_hw()
        self.h = np.zeros((wl.hidden, hm, wm), np.float32)
        self.c = np.zeros((wl.hidden, hm, wm), np.float32)

    def reset(self):
        self.h[...] = 0
        self.c[...] = 0

    def set_state(self, h, c):
        self.h = np.array(h, dtype=np.float32, copy=True)
        self.c = np.array(c, dtype=np.float32, copy=True)

    def step(self, frame: np.ndarray, want_overlay: Optional[bool] = None) -> FrameOutput:
        wl, w = self.wl, self.w
        pre = S.preprocess(frame, wl.net_w, wl.net_h, wl.norm_div, wl.norm_mean, wl.norm_std)
        a = S.round_bf16(pre) if self.mirror else pre     # the first contraction also takes bf16 operands
        enc = []
        for l, s in enumerate(wl.enc_stride):
            a = S.conv3x3(a, w[f"enc_w{l}"], w[f"enc_b{l}"], stride=s, relu=True)
            if self.mirror:
                a = S.round_bf16(a)
            enc.append(a)
        if getattr(wl, "recurrent", True):
            h_in = S.round_bf16(self.h) if self.mirror else self.h
            h2, c2 = S.convlstm_step(a, h_in, self.c, w["lstm_w"], w["lstm_b"])
            self.h, self.c = h2, c2
        else:
            # feed-forward model (the paper's second workload class, Section V-B): the heads read the
            # last encoder output; there is no state to carry
            h2, c2 = enc[-1], np.zeros_like(enc[-1])
        z, p, mask = S.head(h2, w["head_w"], w["head_b"], wl.threshold)
        if wl.conf_mode == "mean_sigmoid":
            conf = S.conf_mean_sigmoid(p)
        else:
            conf = S.conf_gap_linear(h2, w["conf_w"], w["conf_b"])
        cx, cy, n = S.centroids(mask)
        do_ov = wl.overlay if want_overlay is None else want_overlay
        ov = S.overlay(frame, mask, wl.palette) if do_ov else None
        return FrameOutput(pre, enc, h2, c2, z, p, mask, conf, cx, cy, n, ov)
