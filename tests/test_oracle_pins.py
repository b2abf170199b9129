"""Pins for the CPU oracle: closed forms, fixed points, brute force and library special cases.

Each stage of the oracle is compared with something that is not the oracle: exact rational
arithmetic, hand-computed values, mathematical identities, or an independent library
routine (torch CPU in float64) for the special case the stage reduces to.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle

RNG = np.random.default_rng(1234)


# ----------------------------------------------------------------------------- O1 resize
@pytest.mark.parametrize("n_in,n_out", [(i, o) for i in range(1, 40, 3) for o in range(1, 40, 4)]
                         + [(854, 640), (480, 480), (128, 64), (1920, 1280), (1080, 720), (7, 64)])
def test_resize_axis_matches_exact_rational(n_in, n_out):
    i0, i1, fr = oracle.resize_axis(n_in, n_out)
    for o in range(n_out):
        s = (Fraction(2 * o + 1, 2) * n_in) / n_out - Fraction(1, 2)   # (o+1/2)*in/out - 1/2
        s = min(max(s, Fraction(0)), Fraction(n_in - 1))
        lo = s.numerator // s.denominator
        assert i0[o] == lo
        assert i1[o] == min(lo + 1, n_in - 1)
        assert fr[o] == float(s - lo)


def test_resize_identity_scale_is_exact_and_normalise_values():
    img = np.zeros((6, 5, 3), np.uint8)
    img[..., 0] = 0; img[..., 1] = 255; img[..., 2] = 51
    out = oracle.preprocess(img, 5, 6)
    assert np.all(out[0] == np.float32(-2.0))
    assert np.all(out[1] == np.float32(2.0))
    assert np.allclose(out[2], -1.2, atol=1e-6)        # (0.2 - 0.5)/0.25
    img2 = RNG.integers(0, 256, (9, 7, 3), dtype=np.uint8)
    out2 = oracle.preprocess(img2, 7, 9, norm_div=1.0, norm_mean=0.0, norm_std=1.0)
    assert np.array_equal(out2, img2.transpose(2, 0, 1).astype(np.float32))


def test_resize_exact_half_is_block_mean():
    img = RNG.integers(0, 256, (16, 12, 3), dtype=np.uint8)
    out = oracle.preprocess(img, 6, 8, norm_div=1.0, norm_mean=0.0, norm_std=1.0)
    blocks = img.astype(np.float64).reshape(8, 2, 6, 2, 3).mean(axis=(1, 3)).transpose(2, 0, 1)
    assert np.array_equal(out, blocks.astype(np.float32))


def test_resize_constant_image_stays_constant():
    for v in (0, 17, 200, 255):
        img = np.full((37, 53, 3), v, np.uint8)
        out = oracle.preprocess(img, 31, 29)
        assert np.all(out == out.flat[0])
        assert abs(float(out.flat[0]) - ((v / 255.0) - 0.5) / 0.25) < 1e-6


@pytest.mark.parametrize("shape,net", [((48, 85, 3), (64, 48)), ((27, 19, 3), (40, 33)), ((30, 30, 3), (11, 7))])
def test_resize_matches_library_bilinear(shape, net):
    """Half-pixel-centre bilinear without antialiasing is torch's align_corners=False mode."""
    img = RNG.integers(0, 256, shape, dtype=np.uint8)
    nw, nh = net
    out = oracle.preprocess(img, nw, nh, norm_div=1.0, norm_mean=0.0, norm_std=1.0)
    t = torch.from_numpy(img.astype(np.float64)).permute(2, 0, 1)[None]
    ref = F.interpolate(t, size=(nh, nw), mode="bilinear", align_corners=False, antialias=False)[0].numpy()
    assert np.max(np.abs(out - ref)) < 1e-3   # torch derives its weights in floating point
    assert np.max(np.abs(out - ref)) < 2e-4 * 255


def test_preprocess_channel_order_and_pitch():
    img = np.zeros((4, 4, 3), np.uint8); img[..., 0] = 10; img[..., 1] = 20; img[..., 2] = 30
    out = oracle.preprocess(img, 4, 4, 1.0, 0.0, 1.0)
    assert out[0, 0, 0] == 10 and out[1, 0, 0] == 20 and out[2, 0, 0] == 30
    pitch = 16
    buf = np.zeros((4, pitch), np.uint8); buf[:, :12] = img.reshape(4, 12); buf[:, 12:] = 99
    out2 = oracle.preprocess(buf.reshape(-1), 4, 4, 1.0, 0.0, 1.0, pitch=pitch, src_w=4)
    assert np.array_equal(out, out2)


# ------------------------------------------------------------------------------- O2 conv
def _scatter_conv(x, w, b, stride):
    """Independent formulation: every input sample scatters into the outputs it touches."""
    cin, h, wd = x.shape
    cout = w.shape[0]
    ho, wo = (h - 1) // stride + 1, (wd - 1) // stride + 1
    out = np.tile(b.astype(np.float64)[:, None, None], (1, ho, wo))
    for c in range(cin):
        for yi in range(h):
            for xi in range(wd):
                for ky in range(3):
                    for kx in range(3):
                        ny, nx = yi - ky + 1, xi - kx + 1
                        if ny % stride or nx % stride:
                            continue
                        yo, xo = ny // stride, nx // stride
                        if 0 <= yo < ho and 0 <= xo < wo:
                            out[:, yo, xo] += w[:, c, ky, kx].astype(np.float64) * float(x[c, yi, xi])
    return out


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("hw", [(8, 8), (7, 5), (6, 9)])
def test_conv_matches_scatter_brute_force(stride, hw):
    x = RNG.standard_normal((4, *hw)).astype(np.float32)
    w = RNG.standard_normal((3, 4, 3, 3)).astype(np.float32)
    b = RNG.standard_normal(3).astype(np.float32)
    out = oracle.conv3x3(x, w, b, stride=stride)
    ref = _scatter_conv(x, w, b, stride)
    assert out.shape == ref.shape
    assert np.max(np.abs(out - ref)) < 1e-5


@pytest.mark.parametrize("stride", [1, 2])
def test_conv_matches_library_conv2d(stride):
    x = RNG.standard_normal((5, 13, 10)).astype(np.float32)
    w = RNG.standard_normal((6, 5, 3, 3)).astype(np.float32)
    b = RNG.standard_normal(6).astype(np.float32)
    out = oracle.conv3x3(x, w, b, stride=stride, relu=True)
    ref = F.relu(F.conv2d(torch.from_numpy(x).double()[None], torch.from_numpy(w).double(),
                          torch.from_numpy(b).double(), stride=stride, padding=1))[0].numpy()
    assert out.shape == ref.shape
    assert np.max(np.abs(out - ref)) < 1e-5


def test_conv_delta_kernels_fix_orientation():
    x = RNG.standard_normal((1, 6, 7)).astype(np.float32)
    w = np.zeros((1, 1, 3, 3), np.float32); w[0, 0, 1, 1] = 1
    assert np.array_equal(oracle.conv3x3(x, w, None), x)
    # tap (ky=1, kx=2) reads the right neighbour: output is the input shifted left, zero filled
    w = np.zeros((1, 1, 3, 3), np.float32); w[0, 0, 1, 2] = 1
    out = oracle.conv3x3(x, w, None)
    assert np.array_equal(out[0, :, :-1], x[0, :, 1:]) and np.all(out[0, :, -1] == 0)
    # tap (ky=0, kx=1) reads the pixel above: output is the input shifted down
    w = np.zeros((1, 1, 3, 3), np.float32); w[0, 0, 0, 1] = 1
    out = oracle.conv3x3(x, w, None)
    assert np.array_equal(out[0, 1:, :], x[0, :-1, :]) and np.all(out[0, 0, :] == 0)


def test_conv_ones_counts_and_stride2_sizes():
    out = oracle.conv3x3(np.ones((1, 5, 6), np.float32), np.ones((1, 1, 3, 3), np.float32), None)
    assert out[0, 2, 2] == 9 and out[0, 0, 2] == 6 and out[0, 2, 0] == 6 and out[0, 0, 0] == 4 and out[0, 4, 5] == 4
    n = 480
    for expect in (240, 120, 60):
        n = oracle.conv3x3(np.zeros((1, n, 2), np.float32), np.zeros((1, 1, 3, 3), np.float32), None, stride=2).shape[1]
        assert n == expect
    assert oracle.conv3x3(np.zeros((1, 7, 9), np.float32), np.zeros((1, 1, 3, 3), np.float32), None, stride=2).shape == (1, 4, 5)


def test_conv_bias_relu_and_channel_sum():
    x = np.stack([np.full((4, 4), 1.0), np.full((4, 4), -3.0)]).astype(np.float32)
    w = np.zeros((2, 2, 3, 3), np.float32); w[0, 0, 1, 1] = 2; w[0, 1, 1, 1] = 1; w[1, 1, 1, 1] = 1
    b = np.array([0.5, 1.0], np.float32)
    out = oracle.conv3x3(x, w, b, relu=False)
    assert np.all(out[0] == -0.5) and np.all(out[1] == -2.0)
    assert np.all(oracle.conv3x3(x, w, b, relu=True) == 0)


# --------------------------------------------------------------------------- O3 ConvLSTM
def test_convlstm_zero_weights_closed_form():
    ch, cx = 3, 2
    c = RNG.standard_normal((ch, 5, 6)).astype(np.float32)
    h = RNG.standard_normal((ch, 5, 6)).astype(np.float32)
    x = RNG.standard_normal((cx, 5, 6)).astype(np.float32)
    h2, c2 = oracle.convlstm_step(x, h, c, np.zeros((4 * ch, cx + ch, 3, 3), np.float32), np.zeros(4 * ch, np.float32))
    assert np.array_equal(c2, (0.5 * c.astype(np.float64)).astype(np.float32))
    assert np.allclose(h2, 0.5 * np.tanh(c2.astype(np.float64)), atol=1e-7)


def test_convlstm_saturated_gates_and_carry():
    ch, cx = 2, 1
    x = RNG.standard_normal((cx, 4, 4)).astype(np.float32)
    h = np.zeros((ch, 4, 4), np.float32)
    c = RNG.standard_normal((ch, 4, 4)).astype(np.float32)
    w = np.zeros((4 * ch, cx + ch, 3, 3), np.float32)
    for j in range(ch):
        w[2 * ch + j, 0, 1, 1] = 1.0 + j       # g pre-activation = (1+j) * x
    b = np.zeros(4 * ch, np.float32)
    b[0:ch] = 30; b[ch:2 * ch] = -30; b[3 * ch:4 * ch] = 30          # i->1, f->0, o->1
    h2, c2 = oracle.convlstm_step(x, h, c, w, b)
    for j in range(ch):
        g = np.tanh((1.0 + j) * x[0].astype(np.float64))
        assert np.allclose(c2[j], g, atol=1e-6)
        assert np.allclose(h2[j], np.tanh(g), atol=1e-6)
    b[0:ch] = -30; b[ch:2 * ch] = 30                                   # i->0, f->1: state carried
    cc = c.copy(); hh = h.copy()
    for _ in range(20):
        hh, cc = oracle.convlstm_step(x, hh, cc, w, b)
    assert np.allclose(cc, c, atol=1e-6)


def test_convlstm_matches_library_composition_and_gate_order():
    ch, cx, hm, wm = 4, 3, 6, 5
    x = RNG.standard_normal((cx, hm, wm)).astype(np.float32)
    h = RNG.standard_normal((ch, hm, wm)).astype(np.float32) * 0.5
    c = RNG.standard_normal((ch, hm, wm)).astype(np.float32)
    w = (RNG.standard_normal((4 * ch, cx + ch, 3, 3)) * 0.3).astype(np.float32)
    b = RNG.standard_normal(4 * ch).astype(np.float32)
    h2, c2, gates = oracle.convlstm_step(x, h, c, w, b, return_gates=True)
    xin = torch.from_numpy(np.concatenate([x, h])).double()[None]
    pre = F.conv2d(xin, torch.from_numpy(w).double(), torch.from_numpy(b).double(), padding=1)[0]
    i, f, g, o = pre[0:ch], pre[ch:2 * ch], pre[2 * ch:3 * ch], pre[3 * ch:]
    c_ref = torch.sigmoid(f) * torch.from_numpy(c).double() + torch.sigmoid(i) * torch.tanh(g)
    h_ref = torch.sigmoid(o) * torch.tanh(c_ref)
    assert np.max(np.abs(gates - pre.numpy())) < 1e-5
    assert np.max(np.abs(c2 - c_ref.numpy())) < 1e-6
    assert np.max(np.abs(h2 - h_ref.numpy())) < 1e-6


# ------------------------------------------------------------------------------- O4 head
def test_head_sigmoid_identities_and_strict_threshold():
    ch = 3
    hmap = RNG.standard_normal((ch, 4, 5)).astype(np.float32)
    w = RNG.standard_normal((2, ch)).astype(np.float32)
    z, p, m = oracle.head(hmap, w, np.zeros(2, np.float32))
    zn, pn, mn = oracle.head(-hmap, w, np.zeros(2, np.float32))
    assert np.allclose(z, np.einsum("tc,chw->thw", w.astype(np.float64), hmap.astype(np.float64)), atol=1e-6)
    assert np.allclose(p + pn, 1.0, atol=1e-7)
    assert np.all((p > 0) & (p < 1))
    z0, p0, m0 = oracle.head(np.zeros((ch, 2, 2), np.float32), w, np.zeros(2, np.float32))
    assert np.all(p0 == 0.5) and np.all(m0 == 0)          # z == 0 is not above the threshold
    big = np.full((1, 1, 2), 1.0, np.float32)
    zb, pb, mb = oracle.head(big, np.array([[80.0]], np.float32), None)
    assert 0.0 < pb[0, 0, 0] <= 1.0 and mb[0, 0, 0] == 1
    zs, ps, ms = oracle.head(big, np.array([[-80.0]], np.float32), None)
    assert 0.0 < ps[0, 0, 0] < 1e-30 and ms[0, 0, 0] == 0
    # non-default threshold: mask <=> p > thr  <=> z > ln(thr/(1-thr))
    zt, pt, mt = oracle.head(hmap, w, None, thr=0.7)
    far = np.abs(pt - 0.7) > 1e-6
    assert np.array_equal(mt[far], (pt > 0.7)[far].astype(np.uint8))


# --------------------------------------------------------------------- O5 conf + centroid
def test_centroids_hand_computed():
    m = np.zeros((4, 9, 12), np.uint8)
    m[0, 3, 7] = 1                         # single pixel (x=7, y=3)
    m[1, 2:6, 4:11] = 1                    # rectangle x in [4,10], y in [2,5]
    m[3, 0, 0] = 1; m[3, 8, 11] = 1        # two far pixels
    cx, cy, n = oracle.centroids(m)
    assert (cx[0], cy[0], n[0]) == (7.0, 3.0, 1)
    assert (cx[1], cy[1], n[1]) == (7.0, 3.5, 28)
    assert (cx[2], cy[2], n[2]) == (-1.0, -1.0, 0)
    assert (cx[3], cy[3], n[3]) == (5.5, 4.0, 2)


def test_confidences_closed_forms():
    assert np.all(oracle.conf_mean_sigmoid(np.full((3, 5, 4), 0.5, np.float32)) == 0.5)
    p = np.zeros((1, 2, 2), np.float32); p[0, 0, 0] = 1.0
    assert oracle.conf_mean_sigmoid(p)[0] == 0.25
    hmap = np.stack([np.full((3, 4), 2.0), np.full((3, 4), -1.0)]).astype(np.float32)
    w = np.array([[1.0, 1.0], [0.5, 1.0], [0.0, 0.0]], np.float32)
    conf = oracle.conf_gap_linear(hmap, w, np.array([0.0, 0.0, 0.0], np.float32))
    assert abs(conf[0] - 1 / (1 + np.exp(-1.0))) < 1e-7       # GAP of a constant map is the constant
    assert conf[1] == 0.5 and conf[2] == 0.5
    hm2 = np.zeros((1, 2, 2), np.float32); hm2[0, 1, 1] = 4.0      # GAP = 1
    assert abs(oracle.conf_gap_linear(hm2, np.array([[1.0]], np.float32), np.array([-1.0], np.float32))[0] - 0.5) < 1e-7


# ---------------------------------------------------------------------------- O6 overlay
def test_overlay_hand_computed():
    frame = np.zeros((4, 6, 3), np.uint8)
    frame[..., 0] = 10; frame[..., 1] = 200; frame[..., 2] = 255
    pal = [(255, 0, 0), (0, 255, 0)]
    mask = np.zeros((2, 2, 3), np.uint8)
    out = oracle.overlay(frame, mask, pal)
    assert np.array_equal(out[..., :3], frame) and np.all(out[..., 3] == 255)
    mask[0, 0, 0] = 1            # covers source x in {0,1}, y in {0,1}
    out = oracle.overlay(frame, mask, pal)
    # (153*10 + 102*255 + 127)/255 = 27667/255 = 108 ; (153*200+0+127)/255 = 120 ; (153*255+127)/255 = 153
    assert tuple(out[0, 0]) == (108, 120, 153, 255) and tuple(out[1, 1]) == (108, 120, 153, 255)
    assert tuple(out[0, 2]) == (10, 200, 255, 255) and tuple(out[2, 0]) == (10, 200, 255, 255)
    mask[1, 0, 0] = 1            # second tool blended on top of the first, in order
    out = oracle.overlay(frame, mask, pal)
    # r: (153*108+127)/255 = 65 ; g: (153*120 + 102*255 + 127)/255 = 174 ; b: (153*153+127)/255 = 92
    assert tuple(out[0, 0]) == (65, 174, 92, 255)
    same = np.full((2, 2, 3), 77, np.uint8)
    out = oracle.overlay(same, np.ones((1, 1, 1), np.uint8), [(77, 77, 77)])
    assert np.all(out[..., :3] == 77)


def test_overlay_nearest_index_map():
    frame = np.zeros((5, 7, 3), np.uint8)
    mask = np.zeros((1, 2, 3), np.uint8); mask[0, 1, 2] = 1
    out = oracle.overlay(frame, mask, [(255, 255, 255)])
    hit = out[..., 0] > 0
    ys, xs = np.nonzero(hit)
    # my = floor(y*2/5) == 1 <=> y in {3,4};  mx = floor(x*3/7) == 2 <=> x in {5,6}
    assert set(ys) == {3, 4} and set(xs) == {5, 6} and hit.sum() == 4


def test_round_bf16_ties_to_even():
    a = np.array([1.0, 1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e38], np.float32)
    r = oracle.round_bf16(a)
    assert list(r[:5]) == [1.0, 1.0, 1.015625, -1.0, 0.0]


def test_oracle_bf16_rounding_spread():
    """Rounding activations to bf16 moves single elements of the intermediate maps by more than
    2e-2 of the tensor rms while the path's outputs (probabilities) move far less.  This is a
    property of the arithmetic, shown here with the oracle alone; the parity tests of the
    tensor-core path take their intermediate-tensor tolerance from it."""
    import sys, os
    sys.path.insert(0, os.path.dirname(__file__))
    from parity_util import rel_err
    import tt_synth
    wl = tt_synth.workload("cfg4-gain").with_(name="spread", src_w=160, src_h=120, net_w=136, net_h=104)
    w = tt_synth.make_weights(wl)
    fr = tt_synth.make_frames(wl.frame_kind, wl.stream_seed(0), 1, wl.src_w, wl.src_h)[0]
    a = oracle.OraclePipeline(wl, w).step(fr)
    b = oracle.OraclePipeline(wl, w, mirror_bf16=True).step(fr)
    mid = max(rel_err(b.enc[1], a.enc[1]), rel_err(b.h, a.h), rel_err(b.c, a.c))
    assert 1e-2 < mid < 5e-2
    assert rel_err(b.p, a.p) < 1e-2


def test_feed_forward_pipeline_is_the_composition_of_the_pinned_stages_and_stateless():
    """The feed-forward variant (no recurrent cell) must be exactly encoder -> heads: composed here from torch
    conv2d in fp64 and the textbook head formulas, and independent of whatever frames came before."""
    import torch
    import torch.nn.functional as F

    import tt_synth
    from oracle import OraclePipeline
    wl = tt_synth.workload("cfg0-ff-gain").with_(src_w=40, src_h=32, net_w=24, net_h=20, enc_cout=(6, 10), enc_stride=(2, 1),
                                                 hidden=10, n_tools=3, conf_mode="gap_linear")
    w = tt_synth.make_weights(wl)
    assert "lstm_w" not in w and w["head_w"].shape == (3, 10)
    frames = tt_synth.make_frames(wl.frame_kind, wl.stream_seed(0), 3, wl.src_w, wl.src_h)
    ora = OraclePipeline(wl, w)
    outs = [ora.step(frames[t], want_overlay=False) for t in (0, 1, 2)]
    again = ora.step(frames[0], want_overlay=False)
    assert np.array_equal(again.z, outs[0].z) and np.array_equal(again.conf, outs[0].conf)      # no state carried
    x = torch.from_numpy(outs[2].pre.astype(np.float64))[None]
    for l, s in enumerate(wl.enc_stride):
        x = F.relu(F.conv2d(x, torch.from_numpy(w[f"enc_w{l}"].astype(np.float64)), torch.from_numpy(w[f"enc_b{l}"].astype(np.float64)),
                            stride=s, padding=1))
    feat = x[0].numpy()
    z = np.einsum("tc,chw->thw", w["head_w"].astype(np.float64), feat) + w["head_b"].astype(np.float64)[:, None, None]
    assert np.allclose(outs[2].z, z, rtol=1e-5, atol=1e-6)
    conf = 1.0 / (1.0 + np.exp(-(w["conf_w"].astype(np.float64) @ feat.mean(axis=(1, 2)) + w["conf_b"])))
    assert np.allclose(outs[2].conf, conf, rtol=1e-5, atol=1e-6)
    assert np.array_equal(outs[2].mask, (outs[2].z > 0).astype(np.uint8))


def test_render_layers_pins():
    """The multi-layer render load: one layer is the overlay itself; empty masks leave the frame alone; a pixel
    covered by one tool goes through the integer blend once per layer with that layer's colour (by hand)."""
    import oracle
    frame = np.full((4, 6, 3), 0, np.uint8)
    frame[..., 0], frame[..., 1], frame[..., 2] = 10, 200, 77
    pal = [(255, 0, 0), (0, 255, 0), (0, 0, 255)]
    mask = np.zeros((3, 2, 3), np.uint8)
    out = oracle.render_layers(frame, mask, pal, 5)
    assert np.array_equal(out[..., :3], frame) and np.all(out[..., 3] == 255)
    mask[1, 0, 0] = 1                                   # tool 1 covers source pixels x in [0,2), y in [0,2)
    assert np.array_equal(oracle.render_layers(frame, mask, pal, 1), oracle.overlay(frame, mask, pal))
    out = oracle.render_layers(frame, mask, pal, 3)
    rgb = [10, 200, 77]
    for l in range(3):
        c = pal[(1 + l) % 3]                            # layer l paints tool 1 with colour (1 + l) mod 3
        rgb = [(153 * v + 102 * c[k] + 127) // 255 for k, v in enumerate(rgb)]
    assert list(out[0, 0, :3]) == rgb and list(out[1, 1, :3]) == rgb
    assert list(out[0, 2, :3]) == [10, 200, 77] and list(out[3, 5, :3]) == [10, 200, 77]
    # two tools on one pixel: ascending tool order inside a layer
    mask[2, 0, 0] = 1
    out = oracle.render_layers(frame, mask, pal, 2)
    rgb = [10, 200, 77]
    for l in range(2):
        for t in (1, 2):
            c = pal[(t + l) % 3]
            rgb = [(153 * v + 102 * c[k] + 127) // 255 for k, v in enumerate(rgb)]
    assert list(out[0, 0, :3]) == rgb
