"""tt_postprocess_static, the entry point for callers that may not allocate device memory.

Some users of the library run where cudaMalloc is not an option: inside a frame loop that
has promised a fixed memory footprint, or as a plug-in whose buffers come from the host
application's allocator.  For them the library keeps the post-processing scratch in a fixed
array of its own.  This test drives that entry point through the C ABI twice in a row, with
different inputs, and expects bit for bit what tt_postprocess (caller-provided scratch) returns
(both run the same kernels, so nothing may differ), and holds the first call against the CPU
oracle as well; the second call also shows that whatever the first call left in the shared array
does no harm.
It lives in a file that pytest collects last, so a run that stops at the first failure has
already been through every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2402_04466_b200 import binding
from parity_util import assert_close, check_masks, check_reductions_from_own_mask

pytestmark = pytest.mark.gpu


def _case(rng, K, ch, hm, wm, T, dev):
    h = torch.from_numpy((rng.standard_normal((K, hm, wm, ch)) * 0.5).astype(np.float32)).to(dev)
    w = [torch.from_numpy((rng.standard_normal(s) * 0.3).astype(np.float32)).to(dev) for s in ((T, ch), (T,), (T, ch), (T,))]
    return h, w


def _same(a, b):
    """The two entry points run the same kernels on the same inputs: every output must be identical."""
    assert torch.equal(a["masks"], b["masks"])
    assert torch.equal(a["logits"], b["logits"])
    assert torch.equal(a["probs"], b["probs"])
    for ra, rb in zip(a["results"], b["results"]):
        assert np.array_equal(ra["count"], rb["count"])
        assert np.array_equal(ra["cx"], rb["cx"]) and np.array_equal(ra["cy"], rb["cy"])
        assert np.array_equal(ra["conf"], rb["conf"])


def _against_oracle(got, h, hw, hb, cw, cb):
    """The no-allocation entry point held directly against the CPU oracle (fp32 tolerance 1e-4)."""
    for k in range(h.shape[0]):
        hk = np.ascontiguousarray(h[k].cpu().numpy().transpose(2, 0, 1))          # channels-last -> [Ch][Hm][Wm]
        z, p, m = oracle.head(hk, hw.cpu().numpy(), hb.cpu().numpy(), 0.5)
        assert_close(got["logits"][k].cpu().numpy(), z, 1e-4, f"static logits {k}")
        assert_close(got["probs"][k].cpu().numpy(), p, 1e-4, f"static probs {k}")
        gm = got["masks"][k].cpu().numpy()
        check_masks(gm, m, z, 0.0, 1e-3, f"static masks {k}")
        check_reductions_from_own_mask(got["results"][k], gm)
        assert_close(got["results"][k]["conf"], oracle.conf_gap_linear(hk, cw.cpu().numpy(), cb.cpu().numpy()), 1e-4, f"static conf {k}")
        if np.array_equal(gm, m):
            cx, cy, cnt = oracle.centroids(m)
            assert np.array_equal(got["results"][k]["count"], cnt)
            assert np.allclose(got["results"][k]["cx"], cx, atol=1e-4) and np.allclose(got["results"][k]["cy"], cy, atol=1e-4)


def test_static_scratch_matches_caller_scratch_twice_in_a_row(cuda_device):
    rng = np.random.default_rng(5)
    # first call: endoscopy-scale grid, three streams, confidence from the pooled hidden state
    h, (hw, hb, cw, cb) = _case(rng, 3, 128, 60, 80, 7, cuda_device)
    got = binding.postprocess_static(h, True, hw, hb, cw, cb, "gap_linear", 0.5)
    want = binding.postprocess(h, True, hw, hb, cw, cb, "gap_linear", 0.5)
    _same(got, want)
    _against_oracle(got, h, hw, hb, cw, cb)
    assert sum(int(r["count"].sum()) for r in got["results"]) > 0
    # second call straight after, smaller and differently shaped: stale scratch contents must not leak in
    h2, (hw2, hb2, cw2, cb2) = _case(rng, 2, 16, 13, 9, 4, cuda_device)
    got2 = binding.postprocess_static(h2, True, hw2, hb2, None, None, "mean_sigmoid", 0.5)
    want2 = binding.postprocess(h2, True, hw2, hb2, None, None, "mean_sigmoid", 0.5)
    _same(got2, want2)
    # and the first problem again, reusing the caller's output buffers
    again = binding.postprocess_static(h, True, hw, hb, cw, cb, "gap_linear", 0.5, out=got)
    _same(again, want)


def test_static_scratch_rejects_problems_beyond_its_size(cuda_device):
    lib = binding.load_library()
    assert lib.tt_postprocess_scratch_bytes(8, 16, 16, 512, 8) > binding.TT_POSTPROCESS_STATIC_SCRATCH_BYTES
    d = torch.zeros(64, dtype=torch.float32, device=cuda_device)      # never touched: the call is refused up front
    st = lib.tt_postprocess_static(d.data_ptr(), 1, 8, 16, 16, 512, 8, d.data_ptr(), d.data_ptr(), None, None, 0, 0.5,
                                   d.data_ptr(), d.data_ptr(), d.data_ptr(), d.data_ptr(), None)
    assert st == 2
    assert b"scratch" in lib.tt_last_error(None)
    # the largest benchmark shape fits
    assert lib.tt_postprocess_scratch_bytes(8, 90, 160, 256, 7) <= binding.TT_POSTPROCESS_STATIC_SCRATCH_BYTES
