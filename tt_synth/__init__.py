"""Seeded synthetic inputs (frames, weights, workload shapes) for the tool-tracking hot path.

This package only produces *data*: workload shape descriptions, uint8 video frames and
network weights drawn from a counter-based generator.  It contains none of the pipeline's
arithmetic (no resize, convolution, gate math or post-processing) and is imported both by
the CPU oracle's tests and by the CUDA path's tests and benchmark, so that the two sides
see byte-identical inputs without sharing any code of the method itself.
"""
from .rng import splitmix64, uniform01, normal
from .configs import Workload, WORKLOADS, workload
from .frames import make_frames, make_frame
from .weights import make_weights, round_to_bf16

__all__ = [
    "splitmix64", "uniform01", "normal", "Workload", "WORKLOADS", "workload",
    "make_frames", "make_frame", "make_weights", "round_to_bf16",
]
