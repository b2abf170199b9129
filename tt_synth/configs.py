"""Workload shape descriptions (pure data) for the five benchmark configurations.

Index 0 is the tiny fp32 single stream; 1 the endoscopy-scale single stream; 2 is five
concurrent streams of 1; 3 is six streams of 1 with the overlay stage switched on; 4 is the
large scale sweep.  `parity` variants keep every shape but replace the weight standard
deviations by fan-in scaled ones so that the mask logits have O(1) spread (with the nominal
N(0, 0.02) weights nearly every logit lies within 1e-3 of the threshold and masks would be
coin flips).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Tuple

BASE_SEED = 20240204

PALETTE = ((255, 0, 0), (0, 255, 0), (0, 0, 255), (255, 255, 0),
           (255, 0, 255), (0, 255, 255), (255, 128, 0), (128, 128, 128))


@dataclass(frozen=True)
class Workload:
    name: str
    src_w: int
    src_h: int
    net_w: int
    net_h: int
    enc_cout: Tuple[int, ...]
    enc_stride: Tuple[int, ...]
    hidden: int
    n_tools: int
    precision: str            # "fp32" | "bf16"
    conf_mode: str            # "mean_sigmoid" | "gap_linear"
    weight_sigma: float
    frame_kind: str           # "disc" | "endoscopy"
    n_frames: int
    streams: int = 1
    overlay: bool = False
    threshold: float = 0.5
    norm_div: float = 255.0
    norm_mean: float = 0.5
    norm_std: float = 0.25
    gain_corrected: bool = False
    recurrent: bool = True    # False: feed-forward model, the heads read the last encoder output (hidden == enc_cout[-1])
    seed: int = BASE_SEED
    palette: Tuple[Tuple[int, int, int], ...] = field(default=PALETTE)

    @property
    def src_pitch(self) -> int:
        return 3 * self.src_w

    def map_hw(self) -> Tuple[int, int]:
        """(height, width) of the encoder output / recurrent state / mask grid."""
        h, w = self.net_h, self.net_w
        for s in self.enc_stride:
            h = (h + 2 - 3) // s + 1
            w = (w + 2 - 3) // s + 1
        return h, w

    def stream_seed(self, s: int) -> int:
        return self.seed + 1000 * s

    def weight_seed(self) -> int:
        return self.seed + 7

    def parity_variant(self) -> "Workload":
        return replace(self, name=self.name + "-gain", gain_corrected=True)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


_CFG0 = Workload("cfg0", 128, 128, 64, 64, (16,), (1,), 16, 4, "fp32", "mean_sigmoid",
                 0.05, "disc", 8)
_CFG1 = Workload("cfg1", 854, 480, 640, 480, (32, 64, 128), (2, 2, 2), 128, 7, "bf16",
                 "gap_linear", 0.02, "endoscopy", 60)
_CFG2 = replace(_CFG1, name="cfg2", streams=5, n_frames=600)
_CFG3 = replace(_CFG1, name="cfg3", streams=6, n_frames=600, overlay=True)
_CFG4 = Workload("cfg4", 1920, 1080, 1280, 720, (64, 128, 256), (2, 2, 2), 256, 7, "bf16",
                 "gap_linear", 0.02, "endoscopy", 300, streams=8)

WORKLOADS = {w.name: w for w in (_CFG0, _CFG1, _CFG2, _CFG3, _CFG4)}


def feed_forward_variant(wl: Workload) -> Workload:
    """The same encoder and heads without the recurrent cell (a feed-forward segmentation model)."""
    return replace(wl, name=wl.name + "-ff", recurrent=False, hidden=wl.enc_cout[-1])


def workload(name: str) -> Workload:
    """Look up 'cfg0'..'cfg4'; a '-gain' suffix selects the gain-corrected parity variant, a '-ff' suffix
    (before '-gain') the feed-forward variant."""
    if name.endswith("-gain"):
        return workload(name[:-5]).parity_variant()
    if name.endswith("-ff"):
        return feed_forward_variant(workload(name[:-3]))
    return WORKLOADS[name]
