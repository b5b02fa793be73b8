"""Pins for the oracle's NVFP4-granularity statistics (the columns of the paper's Table "stats")."""
import numpy as np

import oracle
from paper_2609_04098_b200 import synth
from tests.golden.load import paper_constants

PC = paper_constants()


def test_error_column_equals_the_quantize_dequantize_route():
    x = synth.config2_activations(0, M=64, K=1024)
    _, g = oracle.calibrate(x)
    st = oracle.stats(x, g)
    grow = oracle.row_scales(64, g=g)
    xh = oracle.dequantize(*oracle.quantize(x, grow), grow)
    xf = synth.bf16_bits_to_f32(x).astype(np.float64)
    assert abs(st["rel_error"] - np.linalg.norm(xf - xh) / np.linalg.norm(xf)) < 1e-6
    assert abs(st["max_over_rms"] - np.abs(xf).max() / np.sqrt((xf ** 2).mean())) < 1e-4 * st["max_over_rms"]
    assert abs(st["kurtosis"] - (xf ** 4).mean() / (xf ** 2).mean() ** 2) < 1e-4 * st["kurtosis"]


def test_gaussian_reference_values():
    segs = synth.make_segments((("w", 256, 0.02),))
    w = synth.weights(0, 21, segs, 2048)
    _, g = oracle.calibrate(w)
    st = oracle.stats(w, g)
    assert abs(st["kurtosis"] - 3.0) < 0.1                         # normal distribution
    assert 4.0 < st["max_over_rms"] < 6.5                           # ~ sqrt(2 ln n) for n = 5e5
    assert st["onehot_share"] < 0.02
    assert PC["w4_error_low"] - 0.02 < st["rel_error"] < PC["w4_error_high"] + 0.006


def test_onehot_threshold_is_nine_sixteenths_of_the_block_energy():
    # block = one value a and fifteen values 1: max/RMS > 3  <=>  a^2 / (a^2 + 15) > 9/16
    assert abs(9.0 / 16.0 - PC["onehot_energy_share"]) < 0.005 and PC["onehot_max_over_rms"] == 3
    def share(a):
        x = synth.f64_to_bf16_bits(np.array([[a] + [1.0] * 15])).reshape(1, 16)
        return oracle.stats(x, 1.0)["onehot_share"]
    a_star = np.sqrt(15 * 9 / 7)                                      # 4.392: energy share exactly 9/16
    assert share(4.5) == 1.0 and share(4.25) == 0.0 and 4.25 < a_star < 4.5
    x = np.zeros((1, 32))
    x[0, 3] = 7.0                                                    # a true one-hot block (max/RMS = 4) and an all-zero one
    st = oracle.stats(synth.f64_to_bf16_bits(x).reshape(1, 32), 1.0)
    assert st["onehot_share"] == 0.5 and abs(st["max_over_rms"] - np.sqrt(32)) < 1e-6


def test_heavy_tailed_activations_look_like_the_papers_rows():
    x = synth.config2_activations(0, M=512, K=5120)
    _, g = oracle.calibrate(x)
    st = oracle.stats(x, g)
    assert st["max_over_rms"] > 40 and st["kurtosis"] > 100          # outliers as in the paper's table (48-368, 39-1809)
    assert 0.03 < st["onehot_share"] < 0.40                          # paper: 5-32 %
    assert 0.005 < st["rel_error"] < 0.12                            # spikes dominate the norm here; paper (per token): 7.5-9.2 %
