"""Stage-level parity: CUDA kernels through the C ABI vs the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
import tt_synth
from paper_2402_04466_b200 import binding
from parity_util import assert_close, check_masks, check_reductions_from_own_mask

pytestmark = pytest.mark.gpu

RNG = np.random.default_rng(77)


def _frames_to_dev(frames, pitch, dev):
    """uint8 [K][H][W][3] -> flat pitched device buffer [K][H*pitch]."""
    K, H, W, _ = frames.shape
    buf = np.full((K, H, pitch), 201, np.uint8)
    buf[:, :, :3 * W] = frames.reshape(K, H, 3 * W)
    return torch.from_numpy(buf.reshape(K, H * pitch)).to(dev)


@pytest.mark.parametrize("src_wh,net_wh,pad,K", [
    ((128, 128), (64, 64), 0, 1),          # exact 2x: block means
    ((854, 480), (640, 480), 0, 2),        # endoscopy scale, identity vertically, unaligned 2562-byte rows
    ((214, 120), (160, 120), 5, 3),        # padded pitch
    ((37, 29), (50, 23), 1, 2),            # upscale x, downscale y, ragged tiles
    ((64, 48), (130, 97), 0, 1),           # 2x upscale, odd outputs (scalar store path)
    ((1920, 1080), (1280, 720), 0, 1),     # scale-sweep size
])
def test_preprocess_matches_oracle(cuda_device, src_wh, net_wh, pad, K):
    (sw, sh), (nw, nh) = src_wh, net_wh
    frames = RNG.integers(0, 256, (K, sh, sw, 3), dtype=np.uint8)
    pitch = 3 * sw + pad
    src = _frames_to_dev(frames, pitch, cuda_device)
    out = binding.preprocess(src, sw, sh, pitch, nw, nh).cpu().numpy()
    for k in range(K):
        ref = oracle.preprocess(frames[k], nw, nh)
        assert_close(out[k], ref, 1e-4, f"preprocess stream {k}")
        assert np.max(np.abs(out[k] - ref)) < 2e-5


def test_preprocess_fixed_points(cuda_device):
    # constant image -> constant output; identity scale -> exactly the normalised input
    img = np.full((1, 40, 52, 3), 93, np.uint8)
    out = binding.preprocess(_frames_to_dev(img, 156, cuda_device), 52, 40, 156, 31, 27).cpu().numpy()
    assert np.all(out == out.flat[0])
    img = RNG.integers(0, 256, (1, 24, 36, 3), dtype=np.uint8)
    out = binding.preprocess(_frames_to_dev(img, 108, cuda_device), 36, 24, 108, 36, 24, 1.0, 0.0, 1.0).cpu().numpy()
    assert np.array_equal(out[0], img[0].transpose(2, 0, 1).astype(np.float32))
    # exact 2x downscale = 2x2 block mean, exact in fp32
    img = RNG.integers(0, 256, (1, 16, 24, 3), dtype=np.uint8)
    out = binding.preprocess(_frames_to_dev(img, 72, cuda_device), 24, 16, 72, 12, 8, 1.0, 0.0, 1.0).cpu().numpy()
    blocks = img[0].astype(np.float64).reshape(8, 2, 12, 2, 3).mean(axis=(1, 3)).transpose(2, 0, 1)
    assert np.array_equal(out[0], blocks.astype(np.float32))


@pytest.mark.parametrize("channels_last", [True, False])
@pytest.mark.parametrize("shape,conf_mode", [
    ((2, 16, 13, 9, 4), "mean_sigmoid"),      # K, Ch, Hm, Wm, T; ragged single tile
    ((3, 128, 60, 80, 7), "gap_linear"),      # endoscopy-scale grid
    ((1, 256, 23, 37, 7), "gap_linear"),      # odd plane, large hidden
    ((2, 64, 8, 8, 8), "mean_sigmoid"),       # exactly one tile, max tools
    ((3, 512, 9, 11, 5), "gap_linear"),       # widest hidden state, plane not a multiple of 4
    ((4, 128, 7, 5, 3), "mean_sigmoid"),      # fewer 4-pixel rounds than warps in the grid; ranges cross streams
    ((8, 256, 31, 33, 8), "gap_linear"),      # 8 streams, max tools, ragged plane
])
def test_postprocess_matches_oracle(cuda_device, channels_last, shape, conf_mode):
    K, ch, hm, wm, T = shape
    h = (RNG.standard_normal((K, ch, hm, wm)) * 0.5).astype(np.float32)
    hw = (RNG.standard_normal((T, ch)) * 0.3).astype(np.float32)
    hb = (RNG.standard_normal(T) * 0.3).astype(np.float32)
    cw = (RNG.standard_normal((T, ch)) * 0.5).astype(np.float32)
    cb = (RNG.standard_normal(T) * 0.3).astype(np.float32)
    dev = cuda_device
    h_dev = torch.from_numpy(h.transpose(0, 2, 3, 1).copy() if channels_last else h).to(dev)
    out = binding.postprocess(h_dev, channels_last, torch.from_numpy(hw).to(dev), torch.from_numpy(hb).to(dev),
                              torch.from_numpy(cw).to(dev), torch.from_numpy(cb).to(dev), conf_mode, 0.5)
    z_g = out["logits"].cpu().numpy(); p_g = out["probs"].cpu().numpy(); m_g = out["masks"].cpu().numpy()
    for k in range(K):
        z, p, m = oracle.head(h[k], hw, hb, 0.5)
        assert_close(z_g[k], z, 1e-4, "logits")
        assert_close(p_g[k], p, 1e-4, "probs")
        check_masks(m_g[k], m, z, 0.0, 1e-3, "masks")
        conf = oracle.conf_mean_sigmoid(p) if conf_mode == "mean_sigmoid" else oracle.conf_gap_linear(h[k], cw, cb)
        r = out["results"][k]
        assert_close(r["conf"], conf, 1e-4, "conf")
        check_reductions_from_own_mask(r, m_g[k])
        cx, cy, n = oracle.centroids(m)
        if np.array_equal(m_g[k], m):
            assert np.array_equal(r["count"], n) and np.array_equal(r["cx"], cx) and np.array_equal(r["cy"], cy)


def test_postprocess_threshold_and_empty_masks(cuda_device):
    dev = cuda_device
    h = np.zeros((1, 4, 5, 6), np.float32); h[0, 0, 2, 3] = 1.0
    hw = np.zeros((2, 4), np.float32); hw[0, 0] = 5.0        # tool 0: single pixel (x=3, y=2); tool 1: z == 0 everywhere
    hb = np.zeros(2, np.float32)
    out = binding.postprocess(torch.from_numpy(h).to(dev), False, torch.from_numpy(hw).to(dev), torch.from_numpy(hb).to(dev))
    r = out["results"][0]
    assert r["count"][0] == 1 and r["cx"][0] == 3.0 and r["cy"][0] == 2.0
    assert r["count"][1] == 0 and r["cx"][1] == -1.0 and r["cy"][1] == -1.0       # z == 0 is not above threshold
    assert np.all(out["probs"].cpu().numpy()[0, 1] == 0.5)
    # threshold 0.7: mask <=> z > ln(7/3)
    hb2 = np.array([0.0, 0.85], np.float32)       # ln(7/3) = 0.8473
    out = binding.postprocess(torch.from_numpy(h).to(dev), False, torch.from_numpy(hw).to(dev), torch.from_numpy(hb2).to(dev),
                              threshold=0.7)
    assert out["results"][0]["count"][1] == 30 and out["results"][0]["count"][0] == 1


@pytest.mark.parametrize("src_wh,grid,pad,K,T", [((854, 480), (60, 80), 0, 2, 7), ((50, 31), (7, 9), 3, 3, 4),
                                                 ((128, 128), (64, 64), 0, 1, 4)])
def test_overlay_is_bit_exact(cuda_device, src_wh, grid, pad, K, T):
    (sw, sh), (hm, wm) = src_wh, grid
    frames = RNG.integers(0, 256, (K, sh, sw, 3), dtype=np.uint8)
    masks = (RNG.random((K, T, hm, wm)) < 0.3).astype(np.uint8)
    pitch = 3 * sw + pad
    out = binding.overlay(_frames_to_dev(frames, pitch, cuda_device), sw, sh, pitch,
                          torch.from_numpy(masks).to(cuda_device), tt_synth.configs.PALETTE).cpu().numpy()
    for k in range(K):
        ref = oracle.overlay(frames[k], masks[k], tt_synth.configs.PALETTE)
        assert np.array_equal(out[k], ref)


@pytest.mark.parametrize("src_wh,grid,pad,K,T,layers", [((214, 120), (15, 20), 0, 2, 7, 3), ((50, 31), (7, 9), 3, 3, 4, 5),
                                                        ((854, 480), (60, 80), 0, 1, 7, 2)])
def test_render_layers_is_bit_exact_in_both_forms(cuda_device, src_wh, grid, pad, K, T, layers):
    """The multi-layer visualisation load against the oracle's layer-by-layer blend: the time-shared form (a block
    per 1024 pixels) and the carved-out form (a few looping blocks) must give the same bytes."""
    (sw, sh), (hm, wm) = src_wh, grid
    frames = RNG.integers(0, 256, (K, sh, sw, 3), dtype=np.uint8)
    masks = (RNG.random((K, T, hm, wm)) < 0.4).astype(np.uint8)
    pitch = 3 * sw + pad
    src = _frames_to_dev(frames, pitch, cuda_device)
    m_dev = torch.from_numpy(masks).to(cuda_device)
    shared = binding.render_layers(src, sw, sh, pitch, m_dev, tt_synth.configs.PALETTE, layers).cpu().numpy()
    carved = binding.render_layers(src, sw, sh, pitch, m_dev, tt_synth.configs.PALETTE, layers, carve_ctas=3).cpu().numpy()
    for k in range(K):
        ref = oracle.render_layers(frames[k], masks[k], tt_synth.configs.PALETTE, layers)
        assert np.array_equal(shared[k], ref)
        assert np.array_equal(carved[k], ref)
