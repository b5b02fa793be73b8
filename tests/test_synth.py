"""The seeded input generator: deterministic, chunk-independent, right statistics."""
import numpy as np

from paper_2609_04098_b200 import synth


def test_deterministic_and_seed_dependent():
    a = synth.prefill_activations(0, 5, 64, 256)
    b = synth.prefill_activations(0, 5, 64, 256)
    c = synth.prefill_activations(1, 5, 64, 256)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    assert a.dtype == np.uint16 and a.shape == (64, 256)


def test_counter_based_prefix_property():
    # element (r, k) depends only on its flat index: a taller tensor starts with the shorter one
    segs_small = synth.make_segments((("w", 16, 0.02),))
    segs_big = synth.make_segments((("w", 48, 0.02),))
    assert np.array_equal(synth.weights(0, 9, segs_big, 128)[:16], synth.weights(0, 9, segs_small, 128))


def test_chunking_does_not_change_values(monkeypatch):
    ref = synth.activations(3, 4, 300, 160, n_hot=3, hot_scale=10.0, spike_p=1e-3)
    monkeypatch.setattr(synth, "_CHUNK", 4096)
    assert np.array_equal(synth.activations(3, 4, 300, 160, n_hot=3, hot_scale=10.0, spike_p=1e-3), ref)


def test_config2_statistics():
    x = synth.bf16_bits_to_f32(synth.config2_activations(0, M=2048, K=5120)).astype(np.float64)
    assert np.abs(x).max() == 2000.0
    spikes = (np.abs(x) == 2000.0).mean()
    assert 0.5e-4 < spikes < 2e-4
    colmed = np.median(np.abs(x), axis=0)          # robust to the +/-2000 spikes
    hot = colmed > 20
    assert hot.sum() == 26                          # 0.5 % of 5120 channels
    assert abs(np.median(colmed[hot]) / np.median(colmed[~hot]) - 100.0) < 10.0


def test_segment_std():
    segs = synth.make_segments(synth.GDN_SEGMENTS)
    assert segs[-1].begin + segs[-1].count == 16480
    small = synth.make_segments((("v", 64, 0.02), ("a", 48, 0.2)))
    w = synth.bf16_bits_to_f32(synth.weights(0, 3, small, 1024)).astype(np.float64)
    assert abs(w[:64].std() - 0.02) < 0.001 and abs(w[64:].std() - 0.2) < 0.01
