"""Pins for the oracle's element codecs (E2M1, E4M3, bf16 rounding).

Nothing here re-types the oracle's own formulas: the checks are brute force
over every code, the tie table that round-to-nearest-even fixes, a library
routine (torch's float8_e4m3fn / bfloat16 casts on CPU), and the numbers the
paper prints (tests/golden/paper_constants.txt).
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from tests.golden.load import paper_constants

PC = paper_constants()
GRID = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]   # the 8 magnitudes a 1-2-1 bit float can hold


def test_e2m1_decode_all_16_codes():
    vals = [oracle.e2m1_decode(c) for c in range(16)]
    assert vals[:8] == GRID
    assert [abs(v) for v in vals[8:]] == GRID
    assert all(np.signbit(np.float32(v)) for v in vals[8:])        # 0x8 is -0
    assert max(vals) == PC["e2m1_top"]


def test_e2m1_roundtrip_all_codes():
    for c in range(16):
        assert oracle.e2m1_encode(oracle.e2m1_decode(c)) == c


def test_e2m1_midpoints_tie_to_even_mantissa():
    # midpoint -> the neighbour whose code has mantissa bit 0
    ties = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}
    for mid, want in ties.items():
        for sign in (1.0, -1.0):
            got = oracle.e2m1_decode(oracle.e2m1_encode(sign * mid))
            assert got == sign * want, (mid, got)
        # one float32 ulp either side goes to the nearer neighbour
        lo = np.nextafter(np.float32(mid), np.float32(0))
        hi = np.nextafter(np.float32(mid), np.float32(10))
        below = max(g for g in GRID if g < mid)
        above = min(g for g in GRID if g > mid)
        assert oracle.e2m1_decode(oracle.e2m1_encode(lo)) == below
        assert oracle.e2m1_decode(oracle.e2m1_encode(hi)) == above


def test_e2m1_nearest_brute_force_and_monotone():
    xs = np.linspace(-7.0, 7.0, 5601, dtype=np.float32)
    prev = -np.inf
    for x in xs:
        got = oracle.e2m1_decode(oracle.e2m1_encode(x))
        best = min(abs(Fraction(float(x)) - Fraction(g)) for g in GRID + [-g for g in GRID])
        assert abs(Fraction(float(x)) - Fraction(got)) == best
        assert got >= prev
        prev = got


def test_e2m1_saturates_and_keeps_sign():
    assert oracle.e2m1_encode(6.0001) == 0x7
    assert oracle.e2m1_encode(-1e30) == 0xF
    assert oracle.e2m1_encode(float("inf")) == 0x7
    assert oracle.e2m1_encode(float("-inf")) == 0xF
    assert oracle.e2m1_encode(-1e-30) == 0x8
    assert oracle.e2m1_encode(-0.0) == 0x8
    assert oracle.e2m1_encode(0.0) == 0x0


def test_e4m3_decode_all_bytes_against_torch():
    raw = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    ref = raw.view(torch.float8_e4m3fn).to(torch.float32).numpy()
    for b in range(256):
        got = oracle.e4m3_decode(b)
        if np.isnan(ref[b]):
            assert np.isnan(got) and (b & 0x7F) == 0x7F
        else:
            assert got == ref[b], b
    assert oracle.e4m3_decode(0x7E) == 448.0
    assert oracle.e4m3_decode(0x01) == 2.0 ** -9
    assert oracle.e4m3_decode(0x08) == 2.0 ** -6
    assert oracle.e4m3_decode(0x38) == 1.0


def test_e4m3_roundtrip_and_midpoints():
    for b in range(0x7F):
        assert oracle.e4m3_encode(oracle.e4m3_decode(b)) == b
    for b in range(0x7E):
        lo, hi = oracle.e4m3_decode(b), oracle.e4m3_decode(b + 1)
        mid = np.float32((lo + hi) / 2)          # exact: both have <= 4 significant bits
        even = b if b % 2 == 0 else b + 1
        assert oracle.e4m3_encode(mid) == even, (b, mid)
        assert oracle.e4m3_encode(np.nextafter(mid, np.float32(0))) == b
        assert oracle.e4m3_encode(np.nextafter(mid, np.float32(1e9))) == b + 1


def test_e4m3_saturation_and_underflow():
    assert oracle.e4m3_encode(448.0) == 0x7E
    assert oracle.e4m3_encode(463.9) == 0x7E
    assert oracle.e4m3_encode(464.0) == 0x7E
    assert oracle.e4m3_encode(1e30) == 0x7E
    assert oracle.e4m3_encode(float("inf")) == 0x7E
    assert oracle.e4m3_encode(2.0 ** -10) == 0x00            # tie between 0 and 2^-9 -> even (0)
    assert oracle.e4m3_encode(np.nextafter(np.float32(2.0 ** -10), np.float32(1))) == 0x01
    assert oracle.e4m3_encode(0.0) == 0x00


def test_e4m3_encode_matches_torch_cast_in_range():
    rng = np.random.default_rng(1)
    v = np.exp(rng.uniform(np.log(2.0 ** -11), np.log(447.9), 20000)).astype(np.float32)
    ref = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([oracle.e4m3_encode(x) for x in v], dtype=np.uint8)
    assert np.array_equal(got, ref)


def test_e4m3_rounding_is_to_nearest_not_up():
    # The paper bounds the re-rounding error of E4M3 local scales by 6.2 %: the
    # half-ulp of a 3-bit mantissa is 2^-4 = 6.25 % of the rounded value; rounding
    # up (or truncating) would allow up to 12.5 %.
    rng = np.random.default_rng(2)
    v = np.exp(rng.uniform(np.log(2.0 ** -6), np.log(448.0), 20000)).astype(np.float32)
    dec = np.array([oracle.e4m3_decode(oracle.e4m3_encode(x)) for x in v], dtype=np.float64)
    rel = np.abs(dec - v) / dec
    assert rel.max() <= 2.0 ** -4
    assert abs(rel.max() - PC["rerounding_error_max"]) < 0.002


def test_f64_to_bf16_matches_torch_on_float32_inputs():
    rng = np.random.default_rng(3)
    v = (rng.standard_normal(50000) * np.exp(rng.uniform(-30, 30, 50000))).astype(np.float32)
    v = np.concatenate([v, np.float32([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40])])
    ref = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = oracle.f64_to_bf16_bits(v.astype(np.float64))
    assert np.array_equal(got, ref)
    assert np.array_equal(oracle.bf16_bits_to_f64(got), torch.from_numpy(v).to(torch.bfloat16).double().numpy())


def test_f64_to_bf16_single_rounding():
    # 1 + 2^-8 + 2^-30 lies just above the tie between 1.0 and 1.0078125: a double
    # rounding through float32 would first drop the 2^-30 and then tie to even (1.0).
    v = 1.0 + 2.0 ** -8 + 2.0 ** -30
    assert oracle.f64_to_bf16_bits(np.array([v]))[0] == 0x3F81
    assert oracle.f64_to_bf16_bits(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80
