"""CPU oracle of the tool-tracking hot path.  TEST INFRASTRUCTURE ONLY.

Plain C (oracle/tt_oracle.c, definition-level nested loops, double accumulation) behind a
numpy/ctypes wrapper, plus a small Python class that chains the stages per frame and keeps
the recurrent state.  Nothing in the CUDA package imports this, and this imports nothing
from the CUDA package.  Only tests, the smoke check and the benchmark's CPU-baseline leg
may use it.

Whole-pipeline parity is unpinned by any published value (the paper prints no tensor);
each stage is pinned separately by tests/test_oracle_*.py.
"""
from .stages import (preprocess, resize_axis, conv3x3, convlstm_step, head, conf_mean_sigmoid,
                     conf_gap_linear, centroids, overlay, render_layers, round_bf16, num_threads, set_threads)
from .pipeline import OraclePipeline, FrameOutput

__all__ = ["preprocess", "resize_axis", "conv3x3", "convlstm_step", "head", "conf_mean_sigmoid",
           "conf_gap_linear", "centroids", "overlay", "render_layers", "round_bf16", "num_threads", "set_threads",
           "OraclePipeline", "FrameOutput"]
