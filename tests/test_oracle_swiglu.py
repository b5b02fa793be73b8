"""Pins for the oracle's silu(gate)*up -> bf16 step (the producer that the quantizer is fused
into).  The paper prescribes no arithmetic for it, so the binary32 sequence in the oracle is a
stated approximation of the textbook definition x*sigmoid(x)*u; the pins bound it against that
definition evaluated in float64 and check its special cases."""
import numpy as np

import oracle
from paper_2609_04098_b200 import synth


def _exact(g, u):
    g = np.asarray(g, np.float64)
    return g / (1.0 + np.exp(-g)) * np.asarray(u, np.float64)


def test_matches_float64_definition_before_rounding():
    rng = np.random.default_rng(0)
    g = np.concatenate([rng.standard_normal(4000) * 3, rng.uniform(-100, 100, 2000)]).astype(np.float32)
    u = (rng.standard_normal(g.size) * 2).astype(np.float32)
    got = np.array([oracle.silu_mul(a, b) for a, b in zip(g, u)], dtype=np.float64)
    want = _exact(g, u)
    big = np.abs(want) > 1e-30
    rel = np.abs(got[big] - want[big]) / np.abs(want[big])
    assert rel.max() < 1e-5            # far below the bf16 half-ulp (2^-9) that follows
    assert np.all(np.abs(got[~big]) < 1e-29)


def test_special_values():
    assert oracle.silu_mul(0.0, 5.0) == 0.0
    assert oracle.silu_mul(100.0, 2.0) == 200.0            # sigmoid saturates to 1
    assert abs(oracle.silu_mul(-100.0, 2.0)) < 1e-30       # and to 0
    assert oracle.silu_mul(1.0, 0.0) == 0.0
    assert oracle.silu_mul(3.0, -1.0) == -oracle.silu_mul(3.0, 1.0)
    xs = np.linspace(-20, 20, 2001, dtype=np.float32)
    ys = np.array([oracle.silu_mul(x, 1.0) for x in xs])
    assert ys.min() > -0.2785 and abs(xs[ys.argmin()] + 1.2785) < 0.03    # the minimum of x*sigmoid(x)


def test_bf16_result_is_the_rounded_definition_almost_everywhere():
    segs = synth.make_segments((("gu", 64, 1.0),))
    gu = synth.weights(3, 77, segs, 512)                     # any bf16 [64, 512]: gate | up, N(0,1)
    h = oracle.swiglu_bf16(gu)
    assert h.shape == (64, 256)
    f = synth.bf16_bits_to_f32(gu).astype(np.float64)
    want = oracle.f64_to_bf16_bits(_exact(f[:, :256], f[:, 256:]))
    same = (h == want)
    assert same.mean() > 0.995
    d = np.abs(oracle.bf16_bits_to_f64(h) - oracle.bf16_bits_to_f64(want))
    ulp = np.abs(oracle.bf16_bits_to_f64((want & np.uint16(0x7FFF)) + np.uint16(1)) - oracle.bf16_bits_to_f64(want & np.uint16(0x7FFF)))
    assert np.all(d <= ulp)
