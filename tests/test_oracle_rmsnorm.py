"""Pins for the oracle's RMSNorm -> bf16 step (the producer of the in-projections' input that
the quantizer is fused into): the float64 definition, special cases, scale invariance."""
import numpy as np

import oracle
from paper_2609_04098_b200 import synth


def _exact(x, w, eps):
    x = x.astype(np.float64)
    return x / np.sqrt((x ** 2).mean(axis=1, keepdims=True) + eps) * w.astype(np.float64)[None, :]


def test_matches_float64_definition_after_rounding():
    x = synth.prefill_activations(0, 70, 24, 5120)                 # two hot channels x50
    w = synth.f64_to_bf16_bits(1.0 + 0.1 * np.sin(np.arange(5120)))
    y = oracle.rmsnorm_bf16(x, w, 1e-6)
    want = oracle.f64_to_bf16_bits(_exact(synth.bf16_bits_to_f32(x), synth.bf16_bits_to_f32(w), 1e-6))
    assert (y == want).mean() > 0.995
    d = np.abs(oracle.bf16_bits_to_f64(y) - oracle.bf16_bits_to_f64(want))
    ulp = np.abs(oracle.bf16_bits_to_f64((want & np.uint16(0x7FFF)) + np.uint16(1)) - oracle.bf16_bits_to_f64(want & np.uint16(0x7FFF)))
    assert np.all(d <= ulp)


def test_special_cases():
    ones = synth.f64_to_bf16_bits(np.ones(64))
    # a constant row normalises to +/-1 (times w)
    x = synth.f64_to_bf16_bits(np.full((2, 64), 3.0) * np.array([[1.0], [-1.0]]))
    y = oracle.bf16_bits_to_f64(oracle.rmsnorm_bf16(x, ones, 0.0))
    assert np.all(y[0] == 1.0) and np.all(y[1] == -1.0)
    # zero row with eps stays zero; scaling x by a power of two changes nothing when eps = 0
    z = oracle.rmsnorm_bf16(np.zeros((1, 32), np.uint16), ones[:32], 1e-6)
    assert np.all((z & 0x7FFF) == 0)
    xr = synth.prefill_activations(1, 71, 4, 256)
    x8 = synth.f64_to_bf16_bits(synth.bf16_bits_to_f32(xr).astype(np.float64) * 8.0).reshape(xr.shape)
    w = synth.f64_to_bf16_bits(np.linspace(0.5, 1.5, 256))
    assert np.array_equal(oracle.rmsnorm_bf16(xr, w, 0.0), oracle.rmsnorm_bf16(x8, w, 0.0))
    # the weight multiplies column-wise
    y1 = oracle.bf16_bits_to_f64(oracle.rmsnorm_bf16(xr, synth.f64_to_bf16_bits(np.ones(256)), 1e-6))
    y2 = oracle.bf16_bits_to_f64(oracle.rmsnorm_bf16(xr, synth.f64_to_bf16_bits(np.full(256, 2.0)), 1e-6))
    assert np.array_equal(y2, 2.0 * y1)
    # unit RMS (before the bf16 rounding of each element, so only approximately)
    assert abs(np.sqrt((y1 ** 2).mean(axis=1)) - 1.0).max() < 5e-3
