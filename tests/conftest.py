import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def cuda_device():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch.device("cuda:0")


def pytest_terminal_summary(terminalreporter):
    """After a GPU run: how many mask pixels differed from the oracle's, and how far from the threshold the
    oracle's logit was at the farthest of them (absolute, and relative to the rms of the frame's logits)."""
    mod = sys.modules.get("test_gpu_pipeline")
    log = getattr(mod, "FLIP_LOG", None) if mod else None
    if not log:
        return
    tr = terminalreporter
    tr.write_sep("-", "mask flips against the oracle")
    for kind, sel in (("fp32 path (tol 1e-4)", [r for r in log if r["tol"] < 1e-3]), ("bf16 path", [r for r in log if r["tol"] >= 1e-3])):
        if not sel:
            continue
        worst = max(sel, key=lambda r: r["margin_rel"])
        tr.write_line(f"{kind}: {len(sel)} frames compared, {sum(r['flips'] for r in sel)} flipped pixels of "
                      f"{sum(r['pixels'] for r in sel)}; largest |z - logit(thr)| at a flip: {max(r['margin'] for r in sel):.3e} "
                      f"absolute, {worst['margin_rel']:.3e} of rms(z) ({worst['tag']}); largest in-band share "
                      f"{max(r['band_frac'] for r in sel):.3%}")
