"""Pins for the oracle's silu(gate)*up -> bf16 step (the producer that the quantizer is fused
into).  The oracle is the textbook definition x*sigmoid(x)*u in double, rounded once to bf16; the
pins are closed forms, special values and a library routine (torch's silu in float64)."""
import numpy as np
import torch

import oracle
from paper_2609_04098_b200 import synth


def test_agrees_with_the_library_silu_in_float64():
    rng = np.random.default_rng(0)
    g = np.concatenate([rng.standard_normal(4000) * 3, rng.uniform(-100, 100, 2000)])
    u = rng.standard_normal(g.size) * 2
    got = np.array([oracle.silu_mul(a, b) for a, b in zip(g, u)])
    want = (torch.nn.functional.silu(torch.from_numpy(g)) * torch.from_numpy(u)).numpy()
    assert np.allclose(got, want, rtol=1e-14, atol=1e-300)


def test_special_values_and_closed_forms():
    assert oracle.silu_mul(0.0, 5.0) == 0.0
    assert oracle.silu_mul(100.0, 2.0) == 200.0            # sigmoid saturates to 1
    assert abs(oracle.silu_mul(-100.0, 2.0)) < 1e-40       # and to 0
    assert oracle.silu_mul(1.0, 0.0) == 0.0
    assert oracle.silu_mul(3.0, -1.0) == -oracle.silu_mul(3.0, 1.0)
    # silu(x) - silu(-x) = x  (sigmoid(x) + sigmoid(-x) = 1)
    for x in (0.3, 1.0, 2.5, 7.0):
        assert abs(oracle.silu_mul(x, 1.0) - oracle.silu_mul(-x, 1.0) - x) < 1e-15
    assert abs(oracle.silu_mul(np.log(3.0), 1.0) - 0.75 * np.log(3.0)) < 1e-15       # sigmoid(ln 3) = 3/4
    xs = np.linspace(-20, 20, 4001)
    ys = np.array([oracle.silu_mul(x, 1.0) for x in xs])
    assert abs(ys.min() + 0.27846) < 1e-4 and abs(xs[ys.argmin()] + 1.2785) < 0.02    # the minimum of x*sigmoid(x)


def test_bf16_result_is_the_definition_rounded_once():
    segs = synth.make_segments((("gu", 64, 1.0),))
    gu = synth.weights(3, 77, segs, 512)                     # any bf16 [64, 512]: gate | up, N(0,1)
    h = oracle.swiglu_bf16(gu)
    assert h.shape == (64, 256)
    f = torch.from_numpy(synth.bf16_bits_to_f32(gu).astype(np.float64))
    want64 = (torch.nn.functional.silu(f[:, :256]) * f[:, 256:]).numpy()
    # rounding through binary32 first could double-round; rounding the double directly must agree
    # with the library's bf16 cast wherever the binary32 intermediate is not a tie
    want = oracle.f64_to_bf16_bits(want64)
    assert np.array_equal(h, want)
    lib = torch.from_numpy(want64).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (h == lib).mean() > 0.9999
    # gate and up are read from the right halves: swapping them changes the result
    swapped = np.concatenate([gu[:, 256:], gu[:, :256]], axis=1)
    assert not np.array_equal(oracle.swiglu_bf16(swapped), h)
