"""B200-native per-frame hot path for K concurrent endoscopy tool-tracking streams.

The compute (preprocess, conv encoder + ConvLSTM step, postprocess, overlay) lives in a
C-ABI shared library built from csrc/ (hand-written CUDA for sm_100a).  This package is
the thin Python binding over it plus host-side measurement helpers; importing it does not
load the library until a binding call needs it, and there is no CPU fallback.
"""
from .stats import latency_summary, percentile, trim_warmup

__all__ = ["latency_summary", "percentile", "trim_warmup"]
