"""End-to-end parity of tt_submit_frames / tt_sync against the CPU oracle on seeded inputs."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import tt_synth
from paper_2402_04466_b200 import binding
from parity_util import assert_close, check_masks, check_reductions_from_own_mask, rel_err, rms_err

pytestmark = pytest.mark.gpu


def _make(wl, K=1, overlay=None, precision=None, timeout_ns=0, plain_launches=False, cta_pairs=False, halo=True,
          fused_pre=False, enc_two_per_sm=True):
    weights = tt_synth.make_weights(wl)
    cfg = binding.make_config(wl, max_streams=K, overlay=overlay, precision=precision, sync_timeout_ns=timeout_ns,
                              plain_launches=plain_launches, cta_pairs=cta_pairs, halo=halo, fused_pre=fused_pre,
                              enc_two_per_sm=enc_two_per_sm)
    ctx = binding.Context(cfg, weights)
    states = [ctx.state_create() for _ in range(K)]
    return ctx, states, weights


def _frames(wl, K, n):
    return [tt_synth.make_frames(wl.frame_kind, wl.stream_seed(s), n, wl.src_w, wl.src_h) for s in range(K)]


# Every frame compared with the oracle leaves a record here; conftest prints the maxima at the end of the
# run (how many mask pixels differ and how far from the threshold the oracle's logit is there), which is
# what the width of the bf16 mask band is derived from.
FLIP_LOG = []


def _compare_frame(ctx, st, res, ref, tol, band, check_tensors=True, tag="", tol_mid=None, max_band_frac=None, log=True):
    """One stream, one frame: every observable of the CUDA path against the oracle's FrameOutput.

    tol bounds the path's float outputs (probabilities, confidences); tol_mid (default: tol)
    bounds the intermediate tensors read through the debug taps.  Masks must agree wherever the
    oracle's logit is at least `band` away from the threshold; max_band_frac bounds the share of
    pixels inside that band (a band that swallows the mask would make the check vacuous).
    """
    stats = {}
    tol_mid = tol if tol_mid is None else tol_mid
    if check_tensors:
        stats["pre"] = assert_close(ctx.debug_tensor(st, "pre"), ref.pre, 1e-4, tag + " pre")
        for l, e in enumerate(ref.enc):
            stats[f"enc{l}"] = assert_close(ctx.debug_tensor(st, f"enc{l}"), e, tol_mid, tag + f" enc{l}")
        if not ctx.cfg.options[binding.TT_OPT_FEED_FORWARD]:          # a feed-forward model carries no state
            stats["c"] = assert_close(ctx.debug_tensor(st, "c"), ref.c, tol_mid, tag + " c")
            stats["h"] = assert_close(ctx.debug_tensor(st, "h"), ref.h, tol_mid, tag + " h")
        stats["logits"] = assert_close(ctx.debug_tensor(st, "logits"), ref.z, tol_mid, tag + " logits")
    stats["prob"] = assert_close(ctx.fetch_probs(res), ref.p, tol, tag + " prob")
    stats["conf"] = assert_close(res["conf"], ref.conf, tol, tag + " conf")
    gm = ctx.fetch_masks(res)
    zthr = float(np.log(ctx.cfg.threshold / (1.0 - ctx.cfg.threshold)))
    stats["band_frac"] = check_masks(gm, ref.mask, ref.z, zthr, band, tag + " mask")
    if max_band_frac is not None:
        assert stats["band_frac"] < max_band_frac, f"{tag}: {stats['band_frac']:.3%} of the pixels lie inside the mask band"
    check_reductions_from_own_mask(res, gm)
    flipped = gm != ref.mask
    flips = int(flipped.sum())
    stats["flips"] = flips
    margin = float(np.abs(ref.z.astype(np.float64) - zthr)[flipped].max()) if flips else 0.0
    z_rms = float(np.sqrt(np.mean(ref.z.astype(np.float64) ** 2)))
    stats["flip_margin"] = margin
    stats["flip_margin_rel"] = margin / max(z_rms, 1e-30)
    if log:
        FLIP_LOG.append({"tag": tag, "flips": flips, "pixels": int(gm.size), "margin": margin, "margin_rel": margin / max(z_rms, 1e-30),
                         "band": band, "band_frac": stats["band_frac"], "tol": tol})
    hm, wm = gm.shape[1], gm.shape[2]
    for t in range(gm.shape[0]):
        n_ref, n_gpu = int(ref.count[t]), int(res["count"][t])
        flips_t = int(flipped[t].sum())
        # every pixel that differs between two masks moves the centroid by at most extent / (size of the smaller mask);
        # with equal masks the centroids are the same number
        if n_ref > 0 and n_gpu > 0:
            slack = flips_t / min(n_ref, n_gpu)
            assert abs(res["cx"][t] - ref.cx[t]) <= slack * wm + 1e-3, (tag, t, flips_t, n_ref)
            assert abs(res["cy"][t] - ref.cy[t]) <= slack * hm + 1e-3, (tag, t, flips_t, n_ref)
    return stats


def test_cfg0_fp32_all_frames(cuda_device):
    """Tiny fp32 single stream: all 8 frames free-running, every tensor at 1e-4."""
    wl = tt_synth.workload("cfg0")
    ctx, (st,), w = _make(wl)
    ora = oracle.OraclePipeline(wl, w)
    frames = _frames(wl, 1, wl.n_frames)[0]
    for t in range(wl.n_frames):
        f = torch.from_numpy(frames[t]).to(cuda_device)
        ctx.submit_frames([f], [st], frame_index=t)
        (res,) = ctx.sync()
        assert res["frame_index"] == t
        _compare_frame(ctx, st, res, ora.step(frames[t]), 1e-4, 1e-3, tag=f"cfg0 t={t}")
    ctx.destroy()


def test_cfg0_gain_variant_has_real_masks(cuda_device):
    wl = tt_synth.workload("cfg0-gain")
    ctx, (st,), w = _make(wl)
    ora = oracle.OraclePipeline(wl, w)
    frames = _frames(wl, 1, 4)[0]
    for t in range(4):
        ctx.submit_frames([torch.from_numpy(frames[t]).to(cuda_device)], [st], frame_index=t)
        (res,) = ctx.sync()
        ref = ora.step(frames[t])
        s = _compare_frame(ctx, st, res, ref, 1e-4, 1e-3, tag=f"cfg0-gain t={t}")
        assert s["band_frac"] < 0.02
    assert 0 < ref.mask.mean() < 1
    ctx.destroy()


def test_fp32_path_stride2_multistream_pinned_host_frames(cuda_device):
    """fp32 kernels on a strided 2-layer encoder, K=3 streams, frames supplied from pinned host memory."""
    wl = tt_synth.workload("cfg0").with_(name="fp32-s2", src_w=150, src_h=110, net_w=100, net_h=76, enc_cout=(8, 24),
                                        enc_stride=(2, 2), hidden=12, n_tools=5, conf_mode="gap_linear",
                                        gain_corrected=True, frame_kind="endoscopy")
    K = 3
    ctx, states, w = _make(wl, K)
    oras = [oracle.OraclePipeline(wl, w) for _ in range(K)]
    frames = _frames(wl, K, 3)
    for t in range(3):
        fs = [torch.from_numpy(frames[k][t]).pin_memory() for k in range(K)]
        ctx.submit_frames(fs, states, frame_index=t)
        res = ctx.sync()
        for k in range(K):
            _compare_frame(ctx, states[k], res[k], oras[k].step(frames[k][t]), 1e-4, 1e-3, tag=f"fp32-s2 k={k} t={t}")
    ctx.destroy()


# Tolerances of the bf16 tensor-core path.  Its float outputs (probabilities, confidences) must
# be within 2e-2 of the oracle.  Intermediate tensors are compared twice: against the oracle
# variant that rounds the same activations to bf16 (max error 2e-2: one bf16 ulp at the bottom
# of a binade is 7.8e-3 and a different accumulation order can flip single roundings, which then
# propagate; rms error 3e-3, which a systematic mistake cannot meet), and against the
# fp32-activation oracle at 5e-2, because bf16 rounding of activations alone moves single
# elements of c, h and the encoder maps by up to 3e-2 of the tensor rms (the oracle shows
# this on its own, see test_oracle_bf16_rounding_spread).
TOL_OUT, TOL_MID_PLAIN, TOL_MIRROR, TOL_MIRROR_RMS = 2e-2, 5e-2, 2e-2, 3e-3
# Mask band of the bf16 path: masks must equal the oracle's wherever the oracle's logit is farther than
# max(1e-3, BAND_REL * rms(z)) from the threshold, and on gain-corrected weights (logits of O(1) spread) less
# than MAX_BAND_FRAC of the pixels may lie inside that band.
BAND_REL, MAX_BAND_FRAC = 2e-2, 0.05


def _run_bf16(cuda_device, wl, K, n_frames, tol_plain=TOL_OUT, tol_mirror=TOL_MIRROR, overlay=False, cta_pairs=False):
    ctx, states, w = _make(wl, K, overlay=overlay, cta_pairs=cta_pairs)
    plain = [oracle.OraclePipeline(wl, w) for _ in range(K)]
    mirror = [oracle.OraclePipeline(wl, w, mirror_bf16=True) for _ in range(K)]
    frames = _frames(wl, K, n_frames)
    worst = {}
    for t in range(n_frames):
        fs = [torch.from_numpy(frames[k][t]).to(cuda_device) for k in range(K)]
        ctx.submit_frames(fs, states, frame_index=t)
        res = ctx.sync()
        for k in range(K):
            ref = plain[k].step(frames[k][t], want_overlay=False)
            # the stated bf16 tolerance against the fp32-activation oracle; masks may differ only
            # where the logit lies within the same tolerance of the threshold
            band = max(1e-3, BAND_REL * float(np.sqrt(np.mean(ref.z.astype(np.float64) ** 2))))
            s = _compare_frame(ctx, states[k], res[k], ref, tol_plain, band, tag=f"{wl.name} plain k={k} t={t}",
                               tol_mid=TOL_MID_PLAIN, max_band_frac=MAX_BAND_FRAC if wl.gain_corrected else None)
            refm = mirror[k].step(frames[k][t], want_overlay=False)
            # both sides rounding the same activations to bf16: only accumulation order and the
            # fast transcendentals differ (a diagnostic: this oracle variant rounds where the kernels
            # round, so no parity claim rests on it)
            bandm = max(1e-3, tol_mirror * float(np.sqrt(np.mean(refm.z.astype(np.float64) ** 2))))
            sm = _compare_frame(ctx, states[k], res[k], refm, tol_mirror, bandm, tag=f"{wl.name} mirror k={k} t={t}", log=False)
            for name, want in (("h", refm.h), ("c", refm.c), ("logits", refm.z)):
                e = rms_err(ctx.debug_tensor(states[k], name), want)
                assert e <= TOL_MIRROR_RMS, f"{wl.name} mirror k={k} t={t} {name}: rms error {e:.3e}"
                worst["rms_" + name] = max(worst.get("rms_" + name, 0), e)
            for key, v in list(s.items()) + [("m_" + a, b) for a, b in sm.items()]:
                worst[key] = max(worst.get(key, 0), v)
            if overlay:
                gm = ctx.fetch_masks(res[k])
                assert np.array_equal(ctx.fetch_overlay(res[k]), oracle.overlay(frames[k][t], gm, wl.palette))
    print(wl.name, {k: (round(v, 6) if isinstance(v, float) else v) for k, v in worst.items()})
    ctx.destroy()
    return worst


def test_bf16_small_ragged_shapes_three_streams(cuda_device):
    """Tensor-core path on a map that is not a multiple of the 16x8 tile, 32- and 64-channel slabs."""
    wl = tt_synth.workload("cfg1-gain").with_(name="bf16-ragged", src_w=200, src_h=150, net_w=176, net_h=136,
                                              enc_cout=(32, 64, 128), hidden=64)
    assert wl.map_hw() == (17, 22)
    _run_bf16(cuda_device, wl, 3, 3)


@pytest.mark.parametrize("shape", [
    dict(src_w=207, src_h=123, net_w=142, net_h=157, enc_cout=(64,), enc_stride=(1,), hidden=32, n_tools=8, conf_mode="mean_sigmoid", K=3, overlay=True),
    dict(src_w=65, src_h=64, net_w=80, net_h=64, enc_cout=(32,), enc_stride=(2,), hidden=128, n_tools=4, conf_mode="mean_sigmoid", K=3, overlay=True),
    dict(src_w=106, src_h=189, net_w=95, net_h=150, enc_cout=(64, 64), enc_stride=(2, 1), hidden=128, n_tools=2, conf_mode="mean_sigmoid", K=3, overlay=False),
    dict(src_w=186, src_h=61, net_w=145, net_h=41, enc_cout=(32, 128), enc_stride=(2, 1), hidden=64, n_tools=4, conf_mode="gap_linear", K=3, overlay=False),
    dict(src_w=133, src_h=130, net_w=84, net_h=151, enc_cout=(32, 128), enc_stride=(1, 1), hidden=128, n_tools=4, conf_mode="mean_sigmoid", K=1, overlay=True),
    dict(src_w=184, src_h=200, net_w=116, net_h=134, enc_cout=(64,), enc_stride=(1,), hidden=64, n_tools=8, conf_mode="mean_sigmoid", K=2, overlay=False),
])
def test_bf16_shapes_drawn_at_random(cuda_device, shape):
    """Shapes drawn once from a seeded generator (widths that are and are not multiples of four, up- and down-scaling,
    one or two layers, every stride mix, 1-8 tools, both confidence modes), kept as a regression set."""
    shape = dict(shape)
    K, overlay = shape.pop("K"), shape.pop("overlay")
    wl = tt_synth.workload("cfg1-gain").with_(name="bf16-drawn", **shape)
    _run_bf16(cuda_device, wl, K, 2, overlay=overlay)


def test_bf16_odd_extents_on_strided_layers(cuda_device):
    """Odd widths and heights at every stride-2 layer: 150x110 -> 75x55 -> 38x28 -> 19x14 (parity views of unequal size)."""
    wl = tt_synth.workload("cfg1-gain").with_(name="bf16-odd", src_w=200, src_h=150, net_w=150, net_h=110,
                                              enc_cout=(32, 64, 128), hidden=32)
    assert wl.map_hw() == (14, 19)
    _run_bf16(cuda_device, wl, 2, 3)


def test_bf16_first_layer_patch_boxes_over_the_image_border(cuda_device):
    """The tensor-core first layer fetches each tile's input patch as one TMA box whose start lies three columns
    left of the halo; with a 148x110 input (rows are 16-byte multiples, nothing else is aligned) the boxes of the
    right and bottom tiles reach past the image and the left and top ones start at negative coordinates."""
    wl = tt_synth.workload("cfg1-gain").with_(name="bf16-border", src_w=200, src_h=150, net_w=148, net_h=110,
                                              enc_cout=(32, 64, 128), hidden=32)
    assert wl.map_hw() == (14, 19)
    _run_bf16(cuda_device, wl, 2, 3)


def test_bf16_first_layer_stride1_on_the_tensor_cores(cuda_device):
    """A stride-1 first layer (18-column patch, 24-column box) with an odd output height."""
    wl = tt_synth.workload("cfg1-gain").with_(name="bf16-first-s1", src_w=96, src_h=72, net_w=64, net_h=45,
                                              enc_cout=(64, 64), enc_stride=(1, 2), hidden=32)
    _run_bf16(cuda_device, wl, 2, 2)


def test_bf16_first_layer_width_outside_the_tensor_core_kernel(cuda_device):
    """A first layer of 96 channels is not covered by the tensor-core first-layer kernel: the fp32 SIMT kernel writes
    the bf16 channels-last map instead, and the next layer runs on 32-channel slabs."""
    wl = tt_synth.workload("cfg1-gain").with_(name="bf16-96", src_w=120, src_h=90, net_w=96, net_h=72,
                                              enc_cout=(96, 64), enc_stride=(2, 2), hidden=32)
    _run_bf16(cuda_device, wl, 2, 2)


def test_bf16_wide_channels_small_map(cuda_device):
    """The scale-sweep channel widths (64/128/256, hidden 256: N = 1024, K = 4608) on a small map."""
    wl = tt_synth.workload("cfg4-gain").with_(name="bf16-wide", src_w=160, src_h=120, net_w=136, net_h=104)
    assert wl.map_hw() == (13, 17)
    _run_bf16(cuda_device, wl, 2, 2)


def test_bf16_cta_pairs_with_an_odd_number_of_tiles(cuda_device):
    """On request the 256-wide ConvLSTM tiles run on CTA pairs (two neighbouring 128-pixel tiles per MMA).  Three
    streams of an 80x40 map give 75 tiles: the last pair has no second tile, its second CTA recomputes the last
    tile and must store nothing.  Checked against the oracle, and bit for bit against single-CTA tiles that add up
    the taps in the same order (one activation box per tap)."""
    wl = tt_synth.workload("cfg1-gain").with_(name="bf16-pairs", src_w=854, src_h=320, net_w=640, net_h=320)
    assert wl.map_hw() == (40, 80)
    _run_bf16(cuda_device, wl, 3, 2, cta_pairs=True)
    K, n = 3, 2
    frames = _frames(wl, K, n)
    outs = []
    for pairs in (True, False):
        ctx, states, _ = _make(wl, K, cta_pairs=pairs, halo=False)
        for t in range(n):
            ctx.submit_frames([torch.from_numpy(frames[k][t]).to(cuda_device) for k in range(K)], states, frame_index=t)
            res = ctx.sync()
        outs.append(([ctx.state_export(s) for s in states], [ctx.fetch_probs(r) for r in res]))
        ctx.destroy()
    for k in range(K):
        assert np.array_equal(outs[0][0][k][0], outs[1][0][k][0]) and np.array_equal(outs[0][0][k][1], outs[1][0][k][1])
        assert np.array_equal(outs[0][1][k], outs[1][1][k])


def test_bf16_postprocess_from_the_fp32_state_still_matches(cuda_device):
    """By default the bf16 path forms the mask and confidence heads on the tensor cores from the bf16 copy of the
    hidden state (every other bf16 test runs that way).  The kernel that reads the fp32 state instead stays
    available; both must match the oracle, and each other within twice the output tolerance."""
    wl = tt_synth.workload("cfg1-gain").with_(name="post-fp32", src_w=214, src_h=120, net_w=160, net_h=120)
    K, n = 2, 2
    frames = _frames(wl, K, n)
    w = tt_synth.make_weights(wl)
    ctxs = []
    for post_tc in (True, False):
        ctx = binding.Context(binding.make_config(wl, max_streams=K, post_tc=post_tc), w)
        ctxs.append((ctx, [ctx.state_create() for _ in range(K)]))
    oras = [oracle.OraclePipeline(wl, w) for _ in range(K)]
    for t in range(n):
        refs = [oras[k].step(frames[k][t], want_overlay=False) for k in range(K)]
        got = []
        for ctx, states in ctxs:
            ctx.submit_frames([torch.from_numpy(frames[k][t]).to(cuda_device) for k in range(K)], states, frame_index=t)
            res = ctx.sync()
            for k in range(K):
                band = max(1e-3, BAND_REL * float(np.sqrt(np.mean(refs[k].z.astype(np.float64) ** 2))))
                _compare_frame(ctx, states[k], res[k], refs[k], TOL_OUT, band, tag=f"post-fp32 k={k} t={t}", tol_mid=TOL_MID_PLAIN,
                               max_band_frac=MAX_BAND_FRAC)
            got.append([(ctx.fetch_probs(r), r["conf"].copy()) for r in res])
        for k in range(K):
            assert_close(got[0][k][0], got[1][k][0], 2 * TOL_OUT, "probabilities of the two postprocess kernels")
            assert_close(got[0][k][1], got[1][k][1], 2 * TOL_OUT, "confidences of the two postprocess kernels")
    for ctx, _ in ctxs:
        ctx.destroy()


def test_bf16_convlstm_one_box_per_tap_still_matches(cuda_device):
    """By default the ConvLSTM fetches one haloed activation patch per channel slab and reads all nine taps from it
    (every other bf16 test runs that way).  The form with one activation box per tap stays available; both must
    match the oracle, and each other up to the order in which the fp32 accumulator adds the taps up."""
    wl = tt_synth.workload("cfg1-gain").with_(name="tapbox", src_w=214, src_h=120, net_w=176, net_h=136, hidden=64)
    K, n = 2, 3
    frames = _frames(wl, K, n)
    outs = []
    for halo in (True, False):
        ctx, states, w = _make(wl, K, halo=halo)
        oras = [oracle.OraclePipeline(wl, w) for _ in range(K)]
        for t in range(n):
            ctx.submit_frames([torch.from_numpy(frames[k][t]).to(cuda_device) for k in range(K)], states, frame_index=t)
            res = ctx.sync()
            for k in range(K):
                ref = oras[k].step(frames[k][t], want_overlay=False)
                band = max(1e-3, BAND_REL * float(np.sqrt(np.mean(ref.z.astype(np.float64) ** 2))))
                _compare_frame(ctx, states[k], res[k], ref, TOL_OUT, band, tag=f"tapbox halo={halo} k={k} t={t}", tol_mid=TOL_MID_PLAIN,
                               max_band_frac=MAX_BAND_FRAC)
        outs.append([ctx.debug_tensor(s, "c") for s in states])
        ctx.destroy()
    for a, b in zip(*outs):
        assert rms_err(a, b) < 1e-3


@pytest.mark.parametrize("shape", [
    dict(src_w=214, src_h=120, net_w=160, net_h=120),                 # one axis resized, ragged tiles
    dict(src_w=203, src_h=157, net_w=132, net_h=100),                 # both axes resized, odd pitch, partial tiles
    dict(src_w=96, src_h=64, net_w=128, net_h=96),                    # up-scaling
    dict(src_w=160, src_h=120, net_w=160, net_h=120, stride1=True),   # no resize, stride-1 first layer
])
def test_bf16_preprocessing_inside_the_first_layer_changes_no_bit(cuda_device, shape):
    """On request the first encoder layer samples the frames itself; against the preprocessing as a kernel of its own
    (which writes the resized fp32 image the layer then reads) every output and the state must be the same bits.
    Stream 1's frames sit at an odd address, and the last frame ends where its buffer ends."""
    shape = dict(shape)
    stride1 = shape.pop("stride1", False)
    wl = tt_synth.workload("cfg1-gain").with_(name="fuse", overlay=True, **shape)
    if stride1:
        wl = wl.with_(enc_stride=(1,) + tuple(wl.enc_stride[1:]))
    K, n = 2, 3
    host = _frames(wl, K, n)
    nbytes = host[0][0].size
    runs = []
    for fused in (True, False):
        ctx, states, _ = _make(wl, K, overlay=True, fused_pre=fused)
        out = []
        for t in range(n):
            bufs = [torch.empty(nbytes + 1, dtype=torch.uint8, device=cuda_device) for _ in range(K)]
            views = []
            for k in range(K):
                v = bufs[k][k:k + nbytes]          # stream 1: odd address, last byte of the frame = last byte of the buffer
                v.copy_(torch.from_numpy(host[k][t]).reshape(-1))
                views.append(v.view(host[k][t].shape))
            ctx.submit_frames(views, states, frame_index=t)
            res = ctx.sync()
            out.append([(ctx.fetch_probs(r), ctx.fetch_masks(r), ctx.fetch_overlay(r), r["conf"].copy(), r["cx"].copy(),
                         ctx.debug_tensor(states[i], "pre"), ctx.debug_tensor(states[i], "enc0")) for i, r in enumerate(res)])
        runs.append((out, [ctx.state_export(s) for s in states]))
        ctx.destroy()
    (a, ha), (b, hb) = runs
    for ta, tb in zip(a, b):
        for ra, rb in zip(ta, tb):
            for va, vb in zip(ra, rb):
                assert np.array_equal(va, vb)
    for (h1, c1), (h2, c2) in zip(ha, hb):
        assert np.array_equal(h1, h2) and np.array_equal(c1, c2)


def test_bf16_encoder_launch_shapes_change_no_bit(cuda_device):
    """The tensor-core encoder layers run two blocks per multiprocessor by default, the 32 -> 64 channel layer with its
    weights resident in shared memory; with one block per multiprocessor (weights streamed with the activations) the
    products are accumulated in the same order, so every output and the state must be the same bits."""
    wl = tt_synth.workload("cfg1-gain").with_(name="shapes", src_w=330, src_h=250, net_w=264, net_h=200, overlay=True)
    K, n = 3, 3
    host = _frames(wl, K, n)
    runs = []
    for two in (True, False):
        ctx, states, _ = _make(wl, K, overlay=True, enc_two_per_sm=two)
        out = []
        for t in range(n):
            ctx.submit_frames([torch.from_numpy(host[k][t]).to(cuda_device) for k in range(K)], states, frame_index=t)
            res = ctx.sync()
            out.append([(ctx.fetch_probs(r), ctx.fetch_masks(r), ctx.fetch_overlay(r), r["conf"].copy(), r["cx"].copy(),
                         ctx.debug_tensor(states[i], "enc1"), ctx.debug_tensor(states[i], "enc2")) for i, r in enumerate(res)])
        runs.append((out, [ctx.state_export(s) for s in states]))
        ctx.destroy()
    (a, ha), (b, hb) = runs
    for ta, tb in zip(a, b):
        for ra, rb in zip(ta, tb):
            for va, vb in zip(ra, rb):
                assert np.array_equal(va, vb)
    for (h1, c1), (h2, c2) in zip(ha, hb):
        assert np.array_equal(h1, h2) and np.array_equal(c1, c2)


def test_bf16_eight_tools_and_mean_sigmoid_confidence(cuda_device):
    """The tensor-core heads with every tool slot in use and the confidence taken as the mean probability (the
    fixed-point probability sums instead of the confidence-head columns)."""
    wl = tt_synth.workload("cfg1-gain").with_(name="bf16-t8", src_w=214, src_h=120, net_w=176, net_h=136, hidden=64, n_tools=8,
                                              conf_mode="mean_sigmoid")
    _run_bf16(cuda_device, wl, 3, 2)


def test_bf16_stride1_encoder_and_overlay(cuda_device):
    wl = tt_synth.workload("cfg1-gain").with_(name="bf16-s1", src_w=96, src_h=72, net_w=64, net_h=48,
                                              enc_cout=(32, 64), enc_stride=(2, 1), hidden=32, overlay=True)
    _run_bf16(cuda_device, wl, 2, 3, overlay=True)


def test_cfg1_gain_endoscopy_scale(cuda_device):
    """854x480 -> 640x480 -> 80x60, hidden 128, gain-corrected weights so masks are real blobs."""
    wl = tt_synth.workload("cfg1-gain")
    worst = _run_bf16(cuda_device, wl, 1, 4)
    assert worst["band_frac"] < 0.05


def test_cfg1_nominal_weights(cuda_device):
    """The configuration as specified (N(0, 0.02) weights): logits are dominated by the head bias."""
    wl = tt_synth.workload("cfg1")
    _run_bf16(cuda_device, wl, 1, 2)


def test_cfg2_five_streams_match_single_stream_runs(cuda_device):
    """K=5 batched launches: each stream equals the oracle, and equals the same stream run alone bit for bit."""
    wl = tt_synth.workload("cfg2-gain")
    K, n = 5, 2
    ctx, states, w = _make(wl, K)
    frames = _frames(wl, K, n)
    oras = [oracle.OraclePipeline(wl, w) for _ in range(K)]
    batched = []
    for t in range(n):
        ctx.submit_frames([torch.from_numpy(frames[k][t]).to(cuda_device) for k in range(K)], states, frame_index=t)
        res = ctx.sync()
        refs = [oras[k].step(frames[k][t], want_overlay=False) for k in range(K)]
        for k in range(K):
            band = max(1e-3, BAND_REL * float(np.sqrt(np.mean(refs[k].z.astype(np.float64) ** 2))))
            _compare_frame(ctx, states[k], res[k], refs[k], TOL_OUT, band, check_tensors=(t == n - 1),
                           tag=f"cfg2 k={k} t={t}", tol_mid=TOL_MID_PLAIN, max_band_frac=MAX_BAND_FRAC)
        batched.append([(ctx.fetch_probs(r), r["conf"].copy(), r["count"].copy()) for r in res])
    h_b = [ctx.state_export(s) for s in states]
    ctx.destroy()
    ctx1, (s1,), _ = _make(wl, 1)
    for k in (0, 3):
        ctx1.state_reset(s1)
        for t in range(n):
            ctx1.submit_frames([torch.from_numpy(frames[k][t]).to(cuda_device)], [s1], frame_index=t)
            (r,) = ctx1.sync()
            assert np.array_equal(ctx1.fetch_probs(r), batched[t][k][0])
            assert np.array_equal(r["conf"], batched[t][k][1]) and np.array_equal(r["count"], batched[t][k][2])
        h1, c1 = ctx1.state_export(s1)
        assert np.array_equal(h1, h_b[k][0]) and np.array_equal(c1, h_b[k][1])
    ctx1.destroy()


def test_teacher_forced_late_frame_and_state_roundtrip(cuda_device):
    """Export the CUDA state after several frames, hand it to the oracle, step both once more."""
    wl = tt_synth.workload("cfg1-gain").with_(name="tf", src_w=214, src_h=120, net_w=160, net_h=120, hidden=64)
    ctx, (st,), w = _make(wl)
    frames = tt_synth.make_frames(wl.frame_kind, wl.stream_seed(0), 7, wl.src_w, wl.src_h, start=300)
    for t in range(6):
        ctx.submit_frames([torch.from_numpy(frames[t]).to(cuda_device)], [st], frame_index=300 + t)
        ctx.sync()
    h, c = ctx.state_export(st)
    assert np.abs(h).max() > 0
    ctx.state_import(st, h, c)
    h2, c2 = ctx.state_export(st)
    assert np.array_equal(h, h2) and np.array_equal(c, c2)
    ora = oracle.OraclePipeline(wl, w)
    ora.set_state(h, c)
    ctx.submit_frames([torch.from_numpy(frames[6]).to(cuda_device)], [st], frame_index=306)
    (res,) = ctx.sync()
    ref = ora.step(frames[6], want_overlay=False)
    band = max(1e-3, BAND_REL * float(np.sqrt(np.mean(ref.z.astype(np.float64) ** 2))))
    _compare_frame(ctx, st, res, ref, TOL_OUT, band, tag="teacher-forced", tol_mid=TOL_MID_PLAIN, max_band_frac=MAX_BAND_FRAC)
    ctx.state_reset(st)
    h0, c0 = ctx.state_export(st)
    assert not h0.any() and not c0.any()
    ctx.destroy()


def test_runs_are_bitwise_reproducible(cuda_device):
    wl = tt_synth.workload("cfg1-gain").with_(name="det", src_w=214, src_h=120, net_w=160, net_h=120)
    K = 2
    frames = _frames(wl, K, 3)
    outs = []
    for rep in range(2):
        ctx, states, _ = _make(wl, K)
        for t in range(3):
            ctx.submit_frames([torch.from_numpy(frames[k][t]).to(cuda_device) for k in range(K)], states)
            res = ctx.sync()
        outs.append(([ctx.state_export(s) for s in states], [ctx.fetch_probs(r) for r in res], [r["conf"] for r in res]))
        ctx.destroy()
    for k in range(K):
        assert np.array_equal(outs[0][0][k][0], outs[1][0][k][0]) and np.array_equal(outs[0][0][k][1], outs[1][0][k][1])
        assert np.array_equal(outs[0][1][k], outs[1][1][k]) and np.array_equal(outs[0][2][k], outs[1][2][k])


def test_graph_replay_matches_plain_launches(cuda_device):
    """A tick replayed from a captured graph must give bit for bit what kernel-by-kernel launches give, while
    the batch size, the set of active streams and the frames' addresses (4-byte aligned or not, which selects
    the overlay variant) change from tick to tick and both submit slots are in use."""
    wl = tt_synth.workload("cfg1-gain").with_(name="graph", src_w=214, src_h=120, net_w=160, net_h=120, overlay=True)
    K, n = 3, 14
    host = _frames(wl, K, n)
    nbytes = host[0][0].size
    # every frame twice on the device: once 4-byte aligned, once at an odd byte offset
    bufs = [[torch.empty(nbytes + 16, dtype=torch.uint8, device=cuda_device) for _ in range(2 * n)] for _ in range(K)]
    shape = host[0][0].shape

    def frame(k, t, odd):
        b = bufs[k][2 * t + int(odd)]
        v = b[1:1 + nbytes] if odd else b[:nbytes]
        v.copy_(torch.from_numpy(host[k][t]).reshape(-1))
        return v.view(shape)

    # which streams take part in tick t, and whether stream 0's frame sits at an odd address
    plan = [((0, 1, 2), False)] * 4 + [((0, 2), False)] * 3 + [((0, 1, 2), True)] * 3 + [((1,), False)] * 2 + [((0, 1, 2), False)] * 2
    assert len(plan) == n
    runs = []
    for plain in (True, False):
        ctx, states, _ = _make(wl, K, overlay=True, plain_launches=plain)
        out = []
        pending = 0
        for t, (who, odd) in enumerate(plan):
            ctx.submit_frames([frame(k, t, odd and k == 0) for k in who], [states[k] for k in who], frame_index=t)
            pending += 1
            if pending == 2:
                r = ctx.sync()
                out.append([(x["frame_index"], ctx.fetch_probs(x), ctx.fetch_overlay(x), x["conf"].copy(), x["cx"].copy(),
                             x["count"].copy()) for x in r])
                pending -= 1
        while pending:
            r = ctx.sync()
            out.append([(x["frame_index"], ctx.fetch_probs(x), ctx.fetch_overlay(x), x["conf"].copy(), x["cx"].copy(),
                         x["count"].copy()) for x in r])
            pending -= 1
        launches, ticks = ctx.get_counters()
        runs.append((out, [ctx.state_export(s) for s in states], ticks, launches))
        ctx.destroy()
    (a, ha, ta, la), (b, hb, tb, lb) = runs
    assert ta == tb == n and la == lb, "replayed ticks must count the launches they contain"
    assert len(a) == len(b) == n
    for ra, rb in zip(a, b):
        assert len(ra) == len(rb)
        for xa, xb in zip(ra, rb):
            assert xa[0] == xb[0]
            for va, vb in zip(xa[1:], xb[1:]):
                assert np.array_equal(va, vb)
    for (h1, c1), (h2, c2) in zip(ha, hb):
        assert np.array_equal(h1, h2) and np.array_equal(c1, c2)


def test_frames_in_a_ring_of_device_buffers_of_any_length(cuda_device):
    """The context remembers which frame pointers its device-side pointer tables hold and skips the table
    refresh when a tick brings a known set.  Frames delivered through rings of 1, 3 and 10 buffer sets (always
    known; known after one round; more sets than tables, so the oldest is replaced every tick) must give
    the same bits as kernel-by-kernel launches from the same rings."""
    wl = tt_synth.workload("cfg1-gain").with_(name="ring", src_w=214, src_h=120, net_w=160, net_h=120, overlay=True)
    K, n = 2, 13
    host = _frames(wl, K, n)
    runs = {}
    for ring, plain in ((1, True), (1, False), (3, False), (10, False), (10, True)):
        bufs = [[torch.empty_like(torch.from_numpy(host[k][0]), device=cuda_device) for _ in range(ring)] for k in range(K)]
        ctx, states, _ = _make(wl, K, overlay=True, plain_launches=plain)
        out = []
        for t in range(n):
            who = (0, 1) if t % 5 != 4 else (1,)        # the batch shrinks now and then: a different pointer set
            for k in who:
                bufs[k][t % ring].copy_(torch.from_numpy(host[k][t]))
            ctx.submit_frames([bufs[k][t % ring] for k in who], [states[k] for k in who], frame_index=t)
            out.append([(x["frame_index"], ctx.fetch_probs(x), ctx.fetch_overlay(x), x["conf"].copy(), x["cx"].copy())
                        for x in ctx.sync()])
        runs[(ring, plain)] = (out, [ctx.state_export(s) for s in states])
        ctx.destroy()
    ref_out, ref_h = runs[(1, True)]
    for key, (out, hs) in runs.items():
        for ra, rb in zip(ref_out, out):
            assert len(ra) == len(rb)
            for xa, xb in zip(ra, rb):
                assert xa[0] == xb[0]
                for va, vb in zip(xa[1:], xb[1:]):
                    assert np.array_equal(va, vb), key
        for (h1, c1), (h2, c2) in zip(ref_h, hs):
            assert np.array_equal(h1, h2) and np.array_equal(c1, c2), key


def test_dependent_launches_change_no_bit(cuda_device):
    """The tensor-core kernels normally start as programmatic dependents of their predecessor (set-up overlapping
    its tail); with stage profiling on every kernel is launched normally behind an event.  Both must give the same
    bits, tick after tick, and stage times must come back in the profiled run."""
    wl = tt_synth.workload("cfg1-gain").with_(name="pdl", src_w=214, src_h=120, net_w=160, net_h=120, overlay=True)
    K = 3
    frames = _frames(wl, K, 4)
    outs = []
    for profiled in (False, True):
        ctx, states, _ = _make(wl, K, overlay=True)
        ctx.set_profiling(profiled)
        per_tick = []
        for t in range(4):
            ctx.submit_frames([torch.from_numpy(frames[k][t]).to(cuda_device) for k in range(K)], states)
            res = ctx.sync()
            per_tick.append([(ctx.fetch_probs(r), ctx.fetch_masks(r), ctx.fetch_overlay(r), r["conf"].copy(), r["count"].copy())
                             for r in res])
        if profiled:
            times = ctx.get_stage_times()
            assert times["convlstm"] > 0 and times["postprocess"] > 0
        outs.append((per_tick, [ctx.state_export(s) for s in states]))
        ctx.destroy()
    (a, ha), (b, hb) = outs
    for ta, tb in zip(a, b):
        for ra, rb in zip(ta, tb):
            for va, vb in zip(ra, rb):
                assert np.array_equal(va, vb)
    for (h1, c1), (h2, c2) in zip(ha, hb):
        assert np.array_equal(h1, h2) and np.array_equal(c1, c2)


@pytest.mark.parametrize("depth", [2, 3])
def test_submits_in_flight_match_serial_execution(cuda_device, depth):
    """Software-pipelined use (`depth` submits in flight: submit t+depth-1 before sync t, pinned host frames over the
    copy stream) must give bit for bit what one-at-a-time execution gives, with results returned oldest first."""
    wl = tt_synth.workload("cfg1-gain").with_(name="pipe", src_w=214, src_h=120, net_w=160, net_h=120, overlay=True)
    K, n = 2, 6
    frames = [[torch.from_numpy(f).pin_memory() for f in fs] for fs in _frames(wl, K, n)]

    def collect(ctx, r):
        return [(x["frame_index"], ctx.fetch_probs(x), ctx.fetch_overlay(x), x["conf"].copy(), x["count"].copy()) for x in r]

    ctx, states, _ = _make(wl, K, overlay=True)
    serial = []
    for t in range(n):
        ctx.submit_frames([frames[k][t] for k in range(K)], states, frame_index=t)
        serial.append(collect(ctx, ctx.sync()))
    h_serial = [ctx.state_export(s) for s in states]
    ctx.destroy()

    ctx, states, _ = _make(wl, K, overlay=True)
    piped = []
    for t in range(depth - 1):
        ctx.submit_frames([frames[k][t] for k in range(K)], states, frame_index=t)
    for t in range(depth - 1, n):
        ctx.submit_frames([frames[k][t] for k in range(K)], states, frame_index=t)
        piped.append(collect(ctx, ctx.sync()))          # results of tick t-depth+1 while the later ones are in flight
    while len(piped) < n:
        piped.append(collect(ctx, ctx.sync()))
    h_piped = [ctx.state_export(s) for s in states]
    ctx.destroy()
    for t in range(n):
        for k in range(K):
            a, b = serial[t][k], piped[t][k]
            assert a[0] == b[0] == t
            assert np.array_equal(a[1], b[1]) and np.array_equal(a[2], b[2])
            assert np.array_equal(a[3], b[3]) and np.array_equal(a[4], b[4])
    for k in range(K):
        assert np.array_equal(h_serial[k][0], h_piped[k][0]) and np.array_equal(h_serial[k][1], h_piped[k][1])


def test_boundary_error_paths(cuda_device):
    wl = tt_synth.workload("cfg0")
    ctx, (st, st2), w = _make(wl, K=2)
    with pytest.raises(binding.TTError) as e:
        ctx.state_create()
    assert e.value.status == 5                                  # admission: only max_streams states
    f = torch.from_numpy(tt_synth.make_frame(wl.frame_kind, 1, 0, wl.src_w, wl.src_h)).to(cuda_device)
    with pytest.raises(binding.TTError) as e:
        ctx.sync()
    assert e.value.status == 6                                  # nothing submitted
    with pytest.raises(binding.TTError) as e:
        ctx.submit_frames([f, f, f], [st, st2, st])
    assert e.value.status == 5                                  # K > max_streams
    with pytest.raises(binding.TTError) as e:
        ctx.submit_frames([f, f], [st, st])
    assert e.value.status == 1                                  # same state twice
    with pytest.raises(binding.TTError) as e:
        ctx.submit_frames([], [])
    assert e.value.status == 1
    assert binding.TT_MAX_IN_FLIGHT == 3
    ctx.submit_frames([f], [st])
    ctx.submit_frames([f], [st2])                               # a second and a third submit may be in flight
    ctx.submit_frames([f], [st])
    with pytest.raises(binding.TTError) as e:
        ctx.submit_frames([f], [st])
    assert e.value.status == 6                                  # but not a fourth
    with pytest.raises(binding.TTError) as e:
        ctx.state_reset(st)
    assert e.value.status == 6
    assert len(ctx.sync()) == 1
    assert len(ctx.sync()) == 1
    with pytest.raises(binding.TTError) as e:
        ctx.state_export(st)
    assert e.value.status == 6                                  # still one in flight
    assert len(ctx.sync()) == 1
    other, (so,), _ = _make(wl)
    with pytest.raises(binding.TTError) as e:
        ctx.submit_frames([f], [so])
    assert e.value.status == 1                                  # foreign state
    other.destroy()
    ctx.destroy()
    # unsupported shapes are refused at create, never routed elsewhere
    bad = tt_synth.workload("cfg1").with_(enc_cout=(32, 48, 128))
    with pytest.raises(binding.TTError) as e:
        binding.Context(binding.make_config(bad), tt_synth.make_weights(bad))
    assert e.value.status == 2


def test_feed_forward_model_bf16_and_fp32(cuda_device):
    """The second workload class of the paper (Section V-B: a feed-forward segmentation network): the same encoder
    and heads without the recurrent cell.  Both precision paths against the oracle; results must not depend on
    earlier frames; state calls are refused."""
    for wl, K, tol, band_rel, tol_mid in (
            (tt_synth.workload("cfg1-ff-gain").with_(name="ff-bf16", src_w=214, src_h=120, net_w=176, net_h=136), 3, TOL_OUT, BAND_REL, TOL_MID_PLAIN),
            (tt_synth.workload("cfg0-ff-gain").with_(name="ff-fp32", src_w=150, src_h=110, net_w=100, net_h=76, enc_cout=(8, 24), enc_stride=(2, 2),
                                                     hidden=24, n_tools=5, conf_mode="gap_linear", frame_kind="endoscopy"), 2, 1e-4, 0.0, 1e-4)):
        ctx, states, w = _make(wl, K)
        assert "lstm_w" not in w
        oras = [oracle.OraclePipeline(wl, w) for _ in range(K)]
        frames = _frames(wl, K, 3)
        first = None
        for t in (0, 1, 2, 0):                                        # frame 0 again at the end: same result as the first time
            ctx.submit_frames([torch.from_numpy(frames[k][t]).to(cuda_device) for k in range(K)], states, frame_index=t)
            res = ctx.sync()
            for k in range(K):
                ref = oras[k].step(frames[k][t], want_overlay=False)
                band = max(1e-3, band_rel * float(np.sqrt(np.mean(ref.z.astype(np.float64) ** 2))))
                _compare_frame(ctx, states[k], res[k], ref, tol, band, tag=f"{wl.name} k={k} t={t}", tol_mid=tol_mid)
            snap = [(ctx.fetch_probs(r), r["conf"].copy(), r["count"].copy()) for r in res]
            if first is None:
                first = snap
        for a, b in zip(first, snap):
            assert all(np.array_equal(x, y) for x, y in zip(a, b))
        with pytest.raises(binding.TTError) as e:
            ctx.state_export(states[0])
        assert e.value.status == 2
        ctx.destroy()
    # hidden must be the last encoder width
    bad = tt_synth.workload("cfg1-ff").with_(hidden=64)
    with pytest.raises(binding.TTError) as e:
        binding.Context(binding.make_config(bad), tt_synth.make_weights(bad.with_(hidden=128)))
    assert e.value.status == 1


def test_two_models_in_the_same_tick_match_their_solo_runs(cuda_device):
    """Heterogeneous concurrency (the paper's Section VI experiment with two different applications on one GPU): a
    recurrent tool-tracking model and a feed-forward segmentation model, each a context with its own CUDA stream,
    are submitted in the same tick and run concurrently.  Each must return bit for bit what it returns alone."""
    wa = tt_synth.workload("cfg1-gain").with_(name="het-rec", src_w=214, src_h=120, net_w=160, net_h=120)
    wb = tt_synth.workload("cfg1-ff-gain").with_(name="het-ff", src_w=320, src_h=200, net_w=256, net_h=160, enc_cout=(32, 64, 64), hidden=64)
    n = 4
    fa, fb = _frames(wa, 2, n), _frames(wb, 3, n)

    def collect(ctx, res):
        return [(ctx.fetch_probs(r), r["conf"].copy(), r["count"].copy(), r["cx"].copy()) for r in res]

    solo = {}
    for name, wl, K, frames in (("a", wa, 2, fa), ("b", wb, 3, fb)):
        ctx, states, _ = _make(wl, K)
        solo[name] = []
        for t in range(n):
            ctx.submit_frames([torch.from_numpy(frames[k][t]).to(cuda_device) for k in range(K)], states, frame_index=t)
            solo[name].append(collect(ctx, ctx.sync()))
        ctx.destroy()
    (ca, sa, _), (cb, sb, w_b) = _make(wa, 2), _make(wb, 3)
    ora_b = oracle.OraclePipeline(wb, w_b)
    for t in range(n):
        ca.submit_frames([torch.from_numpy(fa[k][t]).to(cuda_device) for k in range(2)], sa, frame_index=t)
        cb.submit_frames([torch.from_numpy(fb[k][t]).to(cuda_device) for k in range(3)], sb, frame_index=t)   # both in flight
        ra, rb = ca.sync(), cb.sync()
        for got, want in ((collect(ca, ra), solo["a"][t]), (collect(cb, rb), solo["b"][t])):
            for g, w_ in zip(got, want):
                assert all(np.array_equal(x, y) for x, y in zip(g, w_))
        ref = ora_b.step(fb[0][t], want_overlay=False)
        assert_close(cb.fetch_probs(rb[0]), ref.p, TOL_OUT, f"feed-forward model in a shared tick t={t}")
    ca.destroy()
    cb.destroy()


def test_three_models_on_the_same_frame_as_concurrent_branches(cuda_device):
    """A multi-model stream (the paper's Multi-AI application, Section III-B: three models fed by one video): three
    feed-forward encoder/head sets with different weights read the same frame, each context on its own CUDA stream so
    that the three branches run concurrently.  Every model must match the oracle and its own solo run bit for bit."""
    base = tt_synth.workload("cfg1-ff-gain").with_(src_w=214, src_h=120, net_w=176, net_h=136)
    wls = [base.with_(name=f"multi{j}", seed=base.seed + 31 * (j + 1)) for j in range(3)]
    n = 3
    frames = tt_synth.make_frames(base.frame_kind, base.stream_seed(0), n, base.src_w, base.src_h)
    dev_frames = [torch.from_numpy(f).to(cuda_device) for f in frames]
    streams = [torch.cuda.Stream() for _ in range(3)]
    models = []
    for wl, s in zip(wls, streams):
        w = tt_synth.make_weights(wl)
        ctx = binding.Context(binding.make_config(wl, max_streams=1, cuda_stream=s.cuda_stream), w)
        models.append((wl, w, ctx, ctx.state_create()))
    assert not np.array_equal(models[0][1]["head_w"], models[1][1]["head_w"])      # three different models
    torch.cuda.synchronize()
    together = []
    for t in range(n):
        for _, _, ctx, st in models:
            ctx.submit_frames([dev_frames[t]], [st], frame_index=t)                   # all three in flight
        row = []
        for wl, w, ctx, st in models:
            (res,) = ctx.sync()
            ref = oracle.OraclePipeline(wl, w).step(frames[t], want_overlay=False)
            band = max(1e-3, BAND_REL * float(np.sqrt(np.mean(ref.z.astype(np.float64) ** 2))))
            _compare_frame(ctx, st, res, ref, TOL_OUT, band, tag=f"{wl.name} t={t}", tol_mid=TOL_MID_PLAIN)
            row.append((ctx.fetch_probs(res), res["conf"].copy(), res["count"].copy()))
        together.append(row)
    for j, (wl, w, ctx, st) in enumerate(models):
        for t in range(n):                                                            # the same model alone
            ctx.submit_frames([dev_frames[t]], [st], frame_index=t)
            (res,) = ctx.sync()
            a = (ctx.fetch_probs(res), res["conf"].copy(), res["count"].copy())
            assert all(np.array_equal(x, y) for x, y in zip(a, together[t][j]))
        ctx.destroy()


def test_host_side_sync_timeout_leaves_the_submit_in_flight(cuda_device):
    """Failure detection on the host: with sync_timeout_ns = 1 us the first tt_sync of a scale-sweep-sized tick
    gives up with TT_ERR_TIMEOUT (nothing is lost, the submit stays in flight); repeating the call until it
    succeeds returns exactly what a context without a timeout returns."""
    wl = tt_synth.workload("cfg4-gain")
    fr = torch.from_numpy(tt_synth.make_frame(wl.frame_kind, wl.stream_seed(0), 0, wl.src_w, wl.src_h)).to(cuda_device)
    ctx_ref, (st_ref,), _ = _make(wl)
    ctx_ref.submit_frames([fr], [st_ref])
    (want,) = ctx_ref.sync()
    want_p = ctx_ref.fetch_probs(want)
    ctx, (st,), _ = _make(wl, timeout_ns=1000)
    ctx.submit_frames([fr], [st])                                 # first tick of a context: plain launches, > 100 us of GPU work
    with pytest.raises(binding.TTError) as e:
        ctx.sync()
    assert e.value.status == 7 and "timed out" in str(e.value)
    with pytest.raises(binding.TTError) as e:
        ctx.state_export(st)                                      # the submit is still in flight
    assert e.value.status == 6
    res, tries = None, 0
    while res is None:
        try:
            (res,) = ctx.sync()
        except binding.TTError as err:
            assert err.status == 7
            tries += 1
            assert tries < 10_000_000
    assert np.array_equal(ctx.fetch_probs(res), want_p)
    assert np.array_equal(res["conf"], want["conf"]) and np.array_equal(res["count"], want["count"])
    with pytest.raises(binding.TTError) as e:
        ctx.sync()
    assert e.value.status == 6                                    # nothing left in flight
    ctx.destroy()
    ctx_ref.destroy()


def test_device_side_wait_that_runs_out_is_reported_and_the_context_recovers(cuda_device):
    """Failure detection on the device, in the form that harms nothing: a probe warp waits through the kernels'
    own bounded barrier wait on a barrier that nothing completes, with a limit of about a millisecond.  It gives
    up, records its code and returns; the tick behind it is answered with TT_ERR_DEVICE_STATUS; the tick after
    that runs normally and matches the oracle."""
    wl = tt_synth.workload("cfg1-gain").with_(name="waitprobe", src_w=214, src_h=120, net_w=160, net_h=120, hidden=64)
    ctx, (st,), w = _make(wl)
    ora = oracle.OraclePipeline(wl, w)
    frames = _frames(wl, 1, 4)[0]

    def tick(t):
        ctx.submit_frames([torch.from_numpy(frames[t]).to(cuda_device)], [st], frame_index=t)
        return ctx.sync()[0]

    def check(res, ref, t):
        band = max(1e-3, BAND_REL * float(np.sqrt(np.mean(ref.z.astype(np.float64) ** 2))))
        _compare_frame(ctx, st, res, ref, TOL_OUT, band, tag=f"waitprobe t={t}", tol_mid=TOL_MID_PLAIN)

    check(tick(0), ora.step(frames[0], want_overlay=False), 0)
    ctx.debug_expire_wait(2_000_000)                              # about 1 ms of SM cycles
    with pytest.raises(binding.TTError) as e:
        tick(1)
    assert e.value.status == 8 and "0xa00" in str(e.value).lower()
    ora.step(frames[1], want_overlay=False)                       # the tick itself ran; only its report was poisoned
    with pytest.raises(binding.TTError) as e:
        ctx.sync()
    assert e.value.status == 6                                    # that submit is over
    check(tick(2), ora.step(frames[2], want_overlay=False), 2)   # status word cleared: the context works as before
    check(tick(3), ora.step(frames[3], want_overlay=False), 3)
    with pytest.raises(binding.TTError) as e:
        ctx.debug_expire_wait(0)
    assert e.value.status == 1
    ctx.destroy()


def test_staggered_arrivals_through_the_planner_match_per_stream_runs(cuda_device):
    """Unsynchronised arrivals: four streams with different phases are coalesced by the batch planner into
    ticks of varying composition (virtual time).  Streams are independent, so every stream must see exactly
    the results it gets when it runs alone, whatever batches it shared."""
    wl = tt_synth.workload("cfg1-gain").with_(name="stagger", src_w=214, src_h=120, net_w=160, net_h=120, hidden=64)
    K, n = 4, 10
    period, ms = 16_666_667, 1_000_000
    frames = _frames(wl, K, n)
    dev_frames = [[torch.from_numpy(f).to(cuda_device) for f in fs] for fs in frames]
    sched = binding.Scheduler(max_streams=K, window_ns=2 * ms, deadline_ns=period, max_in_flight=1)
    sids = [sched.admit() for _ in range(K)]
    phases = [0, 100_000, 200_000, 9 * ms]                        # streams 1, 2 arrive while stream 0's tick is in flight
    arrivals = sorted((phases[k] + t * period + (23_000 * ((t * 7 + k) % 5)), k, t) for k in range(K) for t in range(n))
    ctx, states, w_ = _make(wl, K)
    got = {}
    sizes = []
    pending = list(arrivals)
    now, done_at, done_ms = 0, None, 0.0                          # virtual clock; a tick occupies the GPU for 300 us
    while True:
        if done_at is not None and now >= done_at:
            sched.complete(done_ms, done_at)
            done_at = None
        batch, wake = sched.next(now)
        if batch:
            ctx.submit_frames([dev_frames[s][fi] for s, fi, _ in batch], [states[s] for s, _, _ in batch], frame_index=batch[0][1])
            res = ctx.sync()
            done_at, done_ms = now + 300_000, res[0]["gpu_ms"]
            sizes.append(len(batch))
            for (s, fi, _), r in zip(batch, res):
                got[(s, fi)] = (ctx.fetch_probs(r), r["conf"].copy(), r["count"].copy(), r["cx"].copy())
            continue
        times = [t for t in (wake if wake != binding.Scheduler.NEVER else None, pending[0][0] if pending else None, done_at) if t is not None]
        if not times:
            break
        now = max(now, min(times))
        while pending and pending[0][0] <= now:
            _, k, t = pending.pop(0)
            assert sched.arrive(sids[k], t, now)
    st = sched.stats()
    assert st["frames"] == K * n and st["dropped"] == 0 and st["deadline_misses"] == 0
    assert len(got) == K * n and min(sizes) == 1 and max(sizes) >= 2 and st["batches"] < K * n
    ctx.destroy()
    # one of the staggered streams against the oracle, frame by frame: whatever batches its frames shared, the
    # stream must be the oracle's stream (each side carrying its own recurrent state through all n frames)
    ora = oracle.OraclePipeline(wl, w_)
    for t in range(n):
        ref = ora.step(frames[2][t], want_overlay=False)
        p, conf, cnt, cx = got[(2, t)]
        assert_close(p, ref.p, TOL_OUT, f"staggered stream 2 t={t} prob")
        assert_close(conf, ref.conf, TOL_OUT, f"staggered stream 2 t={t} conf")
    ctx1, (s1,), _ = _make(wl, 1)
    for k in range(K):
        ctx1.state_reset(s1)
        for t in range(n):
            ctx1.submit_frames([dev_frames[k][t]], [s1], frame_index=t)
            (r,) = ctx1.sync()
            p, conf, cnt, cx = got[(k, t)]
            assert np.array_equal(ctx1.fetch_probs(r), p) and np.array_equal(r["conf"], conf)
            assert np.array_equal(r["count"], cnt) and np.array_equal(r["cx"], cx)
    ctx1.destroy()
