"""The seeded input generators: determinism, shapes, value ranges, order independence."""
import numpy as np

import tt_synth
from tt_synth.rng import splitmix64


def test_splitmix64_published_vector():
    # First outputs of the reference splitmix64 stream seeded with 0 (state advances by the
    # golden-gamma each call): 0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F.
    g = 0x9E3779B97F4A7C15
    states = np.array([0, g, (2 * g) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64)
    out = splitmix64(states)
    assert [int(x) for x in out] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_counter_based_subranges_agree():
    a = tt_synth.uniform01(5, 9, 100)
    b = tt_synth.uniform01(5, 9, 40, start=60)
    assert np.array_equal(a[60:], b)
    n = tt_synth.normal(3, 1, 200000)
    assert abs(n.mean()) < 0.01 and abs(n.std() - 1.0) < 0.01


def test_frames_are_deterministic_and_shaped():
    wl = tt_synth.workload("cfg1")
    f1 = tt_synth.make_frames(wl.frame_kind, wl.stream_seed(2), 2, 214, 120, start=5)
    f2 = tt_synth.make_frame(wl.frame_kind, wl.stream_seed(2), 6, 214, 120)
    assert f1.shape == (2, 120, 214, 3) and f1.dtype == np.uint8
    assert np.array_equal(f1[1], f2)
    assert not np.array_equal(f1[0], f1[1])
    other = tt_synth.make_frame(wl.frame_kind, wl.stream_seed(3), 6, 214, 120)
    assert not np.array_equal(other, f2)
    d = tt_synth.make_frames("disc", 1, 8, 128, 128)
    assert d.max() == 240 and d.min() >= 32


def test_workload_shapes():
    assert tt_synth.workload("cfg0").map_hw() == (64, 64)
    assert tt_synth.workload("cfg1").map_hw() == (60, 80)
    assert tt_synth.workload("cfg4").map_hw() == (90, 160)
    assert tt_synth.workload("cfg2").streams == 5 and tt_synth.workload("cfg3").overlay


def test_weights_shapes_and_bf16_grid():
    wl = tt_synth.workload("cfg1")
    w = tt_synth.make_weights(wl)
    assert w["lstm_w"].shape == (512, 256, 3, 3) and w["enc_w0"].shape == (32, 3, 3, 3)
    assert w["head_w"].shape == (7, 128) and w["conf_w"].shape == (7, 128)
    for k in ("enc_w0", "enc_w1", "enc_w2", "lstm_w", "head_w", "conf_w"):
        assert np.all((w[k].view(np.uint32) & 0xFFFF) == 0), k      # exactly representable in bf16
    assert abs(float(w["lstm_w"].std()) - 0.02) < 5e-4
    w0 = tt_synth.make_weights(tt_synth.workload("cfg0"))
    assert "conf_w" not in w0 and abs(float(w0["lstm_w"].std()) - 0.05) < 2e-3
    g = tt_synth.make_weights(tt_synth.workload("cfg1-gain"))
    assert abs(float(g["lstm_w"].std()) - (1.0 / (9 * 256)) ** 0.5) < 1e-3
