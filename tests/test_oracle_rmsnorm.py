"""Pins for the oracle's RMSNorm -> bf16 step (the producer of the in-projections' input that
the quantizer is fused into): the library's rms_norm in float64, special cases, scale invariance."""
import numpy as np
import torch

import oracle
from paper_2609_04098_b200 import synth


def test_agrees_with_the_library_rms_norm_in_float64():
    x = synth.prefill_activations(0, 70, 24, 5120)                 # two hot channels x50
    w = synth.f64_to_bf16_bits(1.0 + 0.1 * np.sin(np.arange(5120)))
    y = oracle.rmsnorm_bf16(x, w, 1e-6)
    xf = torch.from_numpy(synth.bf16_bits_to_f32(x).astype(np.float64))
    wf = torch.from_numpy(synth.bf16_bits_to_f32(w).astype(np.float64))
    eps = float(np.float32(1e-6))
    want64 = torch.nn.functional.rms_norm(xf, (5120,), weight=wf, eps=eps).numpy()
    want = oracle.f64_to_bf16_bits(want64)
    # the two float64 evaluations differ in the last bits, which can flip a rounding only at a tie
    assert (y == want).mean() > 0.99999
    d = np.abs(oracle.bf16_bits_to_f64(y) - want64)
    assert np.all(d <= np.abs(want64) * 2.0 ** -8 + 1e-300)


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
    # a large eps dominates: y ~ x * w / sqrt(eps)
    y3 = oracle.bf16_bits_to_f64(oracle.rmsnorm_bf16(xr, synth.f64_to_bf16_bits(np.ones(256)), 1e6))
    xf = synth.bf16_bits_to_f32(xr).astype(np.float64)
    assert np.allclose(y3, xf / np.sqrt((xf ** 2).mean(axis=1, keepdims=True) + 1e6), rtol=2.0 ** -8, atol=1e-30)
