"""Pins for the oracle's scalar codecs (E2M1, E4M3, BF16) -- CPU only.

The C oracle is compared with closed forms, exhaustive sweeps against an
exact-rational brute force (oracle.exact, pure Python on Fractions), library
dtypes as a secondary screen, and hand-picked ties.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import exact


def test_e2m1_magnitude_table():
    # 1 sign / 2 exponent / 1 mantissa bit (paper Section 2) -> these eight magnitudes
    want = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    assert [oracle.e2m1_decode(c) for c in range(8)] == want
    assert [oracle.e2m1_decode(c + 8) for c in range(1, 8)] == [-v for v in want[1:]]
    assert np.signbit(oracle.e2m1_decode(8)) and oracle.e2m1_decode(8) == 0.0
    assert [float(v) for v in exact.E2M1_MAGNITUDES] == want


def test_e2m1_representable_round_trip():
    for c in range(16):
        assert oracle.e2m1_encode(oracle.e2m1_decode(c)) == c


@pytest.mark.parametrize("y,code", [
    (0.25, 0), (0.75, 2), (1.25, 2), (1.75, 4), (2.5, 4), (3.5, 6), (5.0, 6),  # ties -> even code
    (0.2500001, 1), (0.7499999, 1), (5.0000005, 7), (4.9999995, 6),
    (6.0, 7), (6.25, 7), (1e30, 7), (-1e30, 15), (-0.75, 10), (-0.0, 8), (-0.1, 8), (0.0, 0),
])
def test_e2m1_ties_and_saturation(y, code):
    assert oracle.e2m1_encode(y) == code


def test_e2m1_exhaustive_bf16_against_rational_brute_force():
    # every finite BF16 bit pattern, projected directly (rcp = 1)
    bad = []
    for h in range(1 << 16):
        if (h >> 7) & 0xFF == 0xFF:
            continue
        got = oracle.e2m1_encode(oracle.bf16_to_f32(h))
        want = exact.e2m1_code(exact.bf16_bits_to_fraction(h), bool(h >> 15))
        if got != want:
            bad.append((h, got, want))
    assert not bad, bad[:5]


def test_e2m1_matches_ml_dtypes_cast_secondary():
    ml_dtypes = pytest.importorskip("ml_dtypes")
    ys = np.linspace(-7, 7, 2801, dtype=np.float32)
    lib = ys.astype(ml_dtypes.float4_e2m1fn).astype(np.float32)
    ours = np.array([oracle.e2m1_decode(oracle.e2m1_encode(y)) for y in ys], dtype=np.float32)
    assert np.array_equal(lib, ours)


def test_e4m3_pins_and_round_trip():
    assert oracle.e4m3_encode(1.0) == 0x38
    assert oracle.e4m3_encode(0.5) == 0x30
    assert oracle.e4m3_encode(2.0 ** -9) == 0x01
    assert oracle.e4m3_encode(448.0) == 0x7E
    assert oracle.e4m3_decode(0x7E) == 448.0
    for c in range(127):
        v = oracle.e4m3_decode(c)
        assert oracle.e4m3_encode(v) == c
        assert Fraction(v) == exact.E4M3_VALUES[c]
    vals = [oracle.e4m3_decode(c) for c in range(127)]
    assert all(b > a for a, b in zip(vals, vals[1:]))  # strictly increasing codes


def test_e4m3_midpoints_go_to_even_mantissa():
    assert oracle.e4m3_encode(1.0625) == 0x38
    assert oracle.e4m3_encode(1.1875) == 0x3A
    for c in range(126):
        lo, hi = oracle.e4m3_decode(c), oracle.e4m3_decode(c + 1)
        mid = np.float32((lo + hi) / 2)  # exact in FP32
        even = c if c % 2 == 0 else c + 1
        assert oracle.e4m3_encode(mid) == even
        assert oracle.e4m3_encode(np.nextafter(mid, np.float32(0))) == c
        assert oracle.e4m3_encode(np.nextafter(mid, np.float32(1e9))) == c + 1


def test_e4m3_underflow_and_saturation():
    assert oracle.e4m3_encode(2.0 ** -10) == 0x00  # tie between 0 and 2^-9 -> even
    assert oracle.e4m3_encode(np.nextafter(np.float32(2.0 ** -10), np.float32(1))) == 0x01
    assert oracle.e4m3_encode(0.0) == 0x00
    for v in (448.0001, 464.0, 480.0, 1e9):
        assert oracle.e4m3_encode(v) == 0x7E


def test_e4m3_random_against_rational_brute_force_and_library():
    ml_dtypes = pytest.importorskip("ml_dtypes")
    rng = np.random.default_rng(7)
    vs = np.concatenate([
        np.exp(rng.uniform(np.log(2.0 ** -12), np.log(447.0), 4000)),
        rng.uniform(0, 2.0 ** -6, 500),
    ]).astype(np.float32)
    lib = vs.astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    for v, lb in zip(vs, lib):
        got = oracle.e4m3_encode(v)
        assert got == exact.nearest_even_index(Fraction(float(v)), exact.E4M3_VALUES)
        assert got == int(lb)


def test_bf16_decode_and_f64_rounding():
    assert oracle.bf16_to_f32(0x3F80) == 1.0
    assert oracle.bf16_to_f32(0xC000) == -2.0
    assert oracle.bf16_to_f32(0x3DCD) == pytest.approx(0.10009765625, abs=0)
    # one rounding, nearest-even on the 8-bit significand
    assert oracle.f64_to_bf16(1.0) == 0x3F80
    assert oracle.f64_to_bf16(1.0 + 2.0 ** -8) == 0x3F80          # tie -> even
    assert oracle.f64_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -40) == 0x3F81
    assert oracle.f64_to_bf16(1.0 + 3 * 2.0 ** -8) == 0x3F82      # tie -> even
    assert oracle.f64_to_bf16(-3.0) == 0xC040
    assert oracle.f64_to_bf16(0.0) == 0x0000
    # a case where FP64 -> FP32 -> BF16 would round twice and go wrong
    y = 1.0 + 2.0 ** -8 + 2.0 ** -30
    assert oracle.f64_to_bf16(y) == 0x3F81
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(3)
    ys = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    lib = torch.from_numpy(ys).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    ours = oracle.round_bf16(ys.astype(np.float64))
    assert np.array_equal(lib, ours)


def test_round_f32_helper_of_the_rational_model():
    # the rational model's own binary32 rounding, checked against IEEE division of
    # exactly representable operands (correctly rounded by the hardware)
    rng = np.random.default_rng(11)
    for _ in range(3000):
        p, q = int(rng.integers(1, 1 << 24)), int(rng.integers(1, 1 << 24))
        want = Fraction(float(np.float32(p) / np.float32(q)))
        assert exact.round_f32(Fraction(p, q)) == want
    assert exact.round_f32(Fraction(1) + Fraction(1, 1 << 24)) == 1                       # tie -> even
    assert exact.round_f32(Fraction(1) + Fraction(3, 1 << 24)) == Fraction(1) + Fraction(4, 1 << 24)
    assert exact.round_f32(Fraction(3, 1 << 150)) == Fraction(4, 1 << 150)                # subnormal tie
    assert exact.round_f32(Fraction(-5, 3)) == -exact.round_f32(Fraction(5, 3))
