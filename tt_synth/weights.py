"""Seeded network weights (framework-conventional OIHW fp32 arrays) for a Workload.

Nominal: every weight and bias ~ N(0, sigma) with the workload's sigma.  Gain-corrected
parity variant: encoder layers sigma = sqrt(2 / fan_in), ConvLSTM and both heads
sigma = sqrt(1 / fan_in), biases N(0, 0.05) and a constant -0.5 mask-head bias, so logits
have an O(1) spread and bright blobs give connected masks.  For bf16 workloads every weight
tensor (not the biases) is rounded once to bf16 (round-to-nearest-even) and returned as
fp32 holding those values;
both the oracle and the CUDA path consume these already-rounded numbers.
"""
from __future__ import annotations

import math
from typing import Dict

import numpy as np

from .configs import Workload
from .rng import normal


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 -> nearest bf16 (ties to even), returned as fp32."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    rounded = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)
    out = (rounded << np.uint64(16)).astype(np.uint32)
    return out.view(np.float32).reshape(a.shape)


def make_weights(wl: Workload) -> Dict[str, np.ndarray]:
    """Returns enc_w{l}, enc_b{l}, lstm_w, lstm_b (recurrent models), head_w, head_b and (gap_linear) conf_w, conf_b."""
    seed = wl.weight_seed()
    tid = [100]

    def draw(shape, sigma):
        n = int(np.prod(shape))
        v = normal(seed, tid[0], n) * sigma
        tid[0] += 1
        return v.astype(np.float32).reshape(shape)

    bf16 = wl.precision == "bf16"
    out: Dict[str, np.ndarray] = {}
    cin = 3
    for l, cout in enumerate(wl.enc_cout):
        fan_in = 9 * cin
        sw = math.sqrt(2.0 / fan_in) if wl.gain_corrected else wl.weight_sigma
        sb = 0.05 if wl.gain_corrected else wl.weight_sigma
        w = draw((cout, cin, 3, 3), sw)
        b = draw((cout,), sb)
        if bf16:
            w = round_to_bf16(w)
        out[f"enc_w{l}"], out[f"enc_b{l}"] = w, b
        cin = cout
    recurrent = getattr(wl, "recurrent", True)
    ch = wl.hidden if recurrent else cin
    sb = 0.05 if wl.gain_corrected else wl.weight_sigma
    if recurrent:
        fan_in = 9 * (cin + ch)
        sw = math.sqrt(1.0 / fan_in) if wl.gain_corrected else wl.weight_sigma
        w = draw((4 * ch, cin + ch, 3, 3), sw)
        b = draw((4 * ch,), sb)
        if bf16:
            w = round_to_bf16(w)
        out["lstm_w"], out["lstm_b"] = w, b
    # Hidden activations are o*tanh(c') with rms around 0.1-0.3; scale the mask head so
    # logits spread over a few units in the parity variant.  A feed-forward model's heads read
    # ReLU features of O(1) size instead.
    sw = (8.0 if recurrent else 1.0) * math.sqrt(1.0 / ch) if wl.gain_corrected else wl.weight_sigma
    out["head_w"] = draw((wl.n_tools, ch), sw)
    if bf16:
        out["head_w"] = round_to_bf16(out["head_w"])
    hb = draw((wl.n_tools,), sb)
    out["head_b"] = (hb - 0.5).astype(np.float32) if wl.gain_corrected else hb
    if wl.conf_mode == "gap_linear":
        out["conf_w"] = draw((wl.n_tools, ch), sw)
        if bf16:
            out["conf_w"] = round_to_bf16(out["conf_w"])
        out["conf_b"] = draw((wl.n_tools,), sb)
    return out
