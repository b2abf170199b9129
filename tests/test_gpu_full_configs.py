"""Parity at the full benchmark sizes: cfg1 free-running over all 60 frames, cfg2 teacher-forced at
late frames, cfg3 with the overlay, cfg4 at the scale-sweep size (oracle on K=2; K=8 checked for
bitwise agreement with the K=2 launches)."""
import numpy as np
import pytest
import torch

import oracle
import tt_synth
from paper_2402_04466_b200 import binding
from parity_util import assert_close
from test_gpu_pipeline import BAND_REL, MAX_BAND_FRAC, TOL_MID_PLAIN, TOL_OUT, _compare_frame, _make

pytestmark = pytest.mark.gpu


def _band(ref):
    return max(1e-3, BAND_REL * float(np.sqrt(np.mean(ref.z.astype(np.float64) ** 2))))


def test_cfg1_sixty_frames_free_running(cuda_device):
    wl = tt_synth.workload("cfg1-gain")
    ctx, (st,), w = _make(wl)
    ora = oracle.OraclePipeline(wl, w)
    worst = 0.0
    for t in range(wl.n_frames):
        fr = tt_synth.make_frame(wl.frame_kind, wl.stream_seed(0), t, wl.src_w, wl.src_h)
        ctx.submit_frames([torch.from_numpy(fr).to(cuda_device)], [st], frame_index=t)
        (res,) = ctx.sync()
        ref = ora.step(fr, want_overlay=False)
        s = _compare_frame(ctx, st, res, ref, TOL_OUT, _band(ref), check_tensors=(t % 15 == 14 or t == 0),
                           tag=f"cfg1 t={t}", tol_mid=TOL_MID_PLAIN, max_band_frac=MAX_BAND_FRAC)
        worst = max(worst, s["prob"])
    print("cfg1 60 frames: worst prob error", worst)
    ctx.destroy()


def test_cfg2_teacher_forced_late_frames(cuda_device):
    """600 frames per stream on the GPU (frames cycle through a ring of 16); at frames 100, 300 and 599 the
    exported state of two of the five streams is handed to the oracle, which takes the same single step."""
    wl = tt_synth.workload("cfg2-gain")
    K, R = wl.streams, 16
    ctx, states, w = _make(wl, K)
    ring = [[tt_synth.make_frame(wl.frame_kind, wl.stream_seed(k), t, wl.src_w, wl.src_h) for t in range(R)] for k in range(K)]
    dev = [[torch.from_numpy(f).to(cuda_device) for f in ring[k]] for k in range(K)]
    checks = {100, 300, 599}
    for t in range(600):
        prev = {k: ctx.state_export(states[k]) for k in (1, 4)} if t in checks else None
        ctx.submit_frames([dev[k][t % R] for k in range(K)], states, frame_index=t)
        res = ctx.sync()
        assert all(r["frame_index"] == t for r in res)
        if prev is not None:
            for k in (1, 4):
                ora = oracle.OraclePipeline(wl, w)
                ora.set_state(*prev[k])
                ref = ora.step(ring[k][t % R], want_overlay=False)
                _compare_frame(ctx, states[k], res[k], ref, TOL_OUT, _band(ref), tag=f"cfg2 k={k} t={t}", tol_mid=TOL_MID_PLAIN,
                               max_band_frac=MAX_BAND_FRAC)
                h, c = ctx.state_export(states[k])
                assert np.isfinite(h).all() and np.isfinite(c).all()
    ctx.destroy()


def test_cfg3_six_streams_with_overlay(cuda_device):
    """Six streams with the overlay stage, 32 free-running frames.  The oracle follows two of the six streams
    through all 32 frames (each side evolving its own recurrent state from zero); the overlay of every stream is
    checked bit for bit against the oracle's blend of the masks the CUDA path produced, on every frame."""
    wl = tt_synth.workload("cfg3-gain")
    K, n, followed = wl.streams, 32, (0, 4)
    assert K == 6 and wl.overlay
    ctx, states, w = _make(wl, K)
    oras = {k: oracle.OraclePipeline(wl, w) for k in followed}
    for t in range(n):
        frames = [tt_synth.make_frame(wl.frame_kind, wl.stream_seed(k), t, wl.src_w, wl.src_h) for k in range(K)]
        ctx.submit_frames([torch.from_numpy(f).to(cuda_device) for f in frames], states, frame_index=t)
        res = ctx.sync()
        for k in range(K):
            gm = ctx.fetch_masks(res[k])
            if k in followed or t % 8 == 0:
                assert np.array_equal(ctx.fetch_overlay(res[k]), oracle.overlay(frames[k], gm, wl.palette))   # integer blend: bit-exact
            if k in followed:
                ref = oras[k].step(frames[k], want_overlay=False)
                _compare_frame(ctx, states[k], res[k], ref, TOL_OUT, _band(ref), check_tensors=(t in (1, n - 1)),
                               tag=f"cfg3 k={k} t={t}", tol_mid=TOL_MID_PLAIN, max_band_frac=MAX_BAND_FRAC)
                if np.array_equal(gm, ref.mask):
                    assert np.array_equal(ctx.fetch_overlay(res[k]), oracle.overlay(frames[k], ref.mask, wl.palette))
    ctx.destroy()


def test_cfg4_scale_sweep_size(cuda_device):
    """1920x1080 -> 1280x720 -> 160x90, hidden 256.  The oracle follows two streams for three frames; the
    K=8 launch configuration that bench.py times must reproduce those two streams bit for bit."""
    wl = tt_synth.workload("cfg4-gain")
    n = 3
    frames = [[tt_synth.make_frame(wl.frame_kind, wl.stream_seed(k), t, wl.src_w, wl.src_h) for t in range(n)] for k in range(8)]
    ctx, states, w = _make(wl, 2)
    oras = [oracle.OraclePipeline(wl, w) for _ in range(2)]
    small = []
    for t in range(n):
        ctx.submit_frames([torch.from_numpy(frames[k][t]).to(cuda_device) for k in range(2)], states, frame_index=t)
        res = ctx.sync()
        for k in range(2):
            ref = oras[k].step(frames[k][t], want_overlay=False)
            _compare_frame(ctx, states[k], res[k], ref, TOL_OUT, _band(ref), check_tensors=(t == n - 1), tag=f"cfg4 k={k} t={t}",
                           tol_mid=TOL_MID_PLAIN, max_band_frac=MAX_BAND_FRAC)
        small.append([(ctx.fetch_probs(r), r["conf"].copy(), r["count"].copy(), r["cx"].copy()) for r in res])
    h_small = [ctx.state_export(s) for s in states]
    ctx.destroy()

    ctx8, states8, _ = _make(wl, 8)
    for t in range(n):
        ctx8.submit_frames([torch.from_numpy(frames[k][t]).to(cuda_device) for k in range(8)], states8, frame_index=t)
        res = ctx8.sync()
        for k in range(2):
            assert np.array_equal(ctx8.fetch_probs(res[k]), small[t][k][0])
            assert np.array_equal(res[k]["conf"], small[t][k][1]) and np.array_equal(res[k]["count"], small[t][k][2])
            assert np.array_equal(res[k]["cx"], small[t][k][3])
        for k in range(2, 8):
            p = ctx8.fetch_probs(res[k])
            assert np.isfinite(p).all() and (p > 0).all() and (p < 1).all()
    for k in range(2):
        h8, c8 = ctx8.state_export(states8[k])
        assert np.array_equal(h8, h_small[k][0]) and np.array_equal(c8, h_small[k][1])
    ctx8.destroy()
