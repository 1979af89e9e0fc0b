"""Pins for the oracle's MXFP4 quantizer and linear -- CPU only."""
from fractions import Fraction

import numpy as np
import torch

import oracle

GRID = [0, 0.5, 1, 1.5, 2, 3, 4, 6]


def bits(values) -> np.ndarray:
    t = torch.tensor(np.asarray(values, dtype=np.float64), dtype=torch.float64)
    h = t.to(torch.bfloat16)
    assert torch.equal(h.to(torch.float64), t), "test input not representable in BF16"
    return h.view(torch.int16).numpy().view(np.uint16)


def rand_bits(rng, shape, scale=1.0) -> np.ndarray:
    return torch.from_numpy(rng.standard_normal(shape) * scale).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def nibbles(q):
    out = np.empty((q.shape[0], q.shape[1] * 2), np.uint8)
    out[:, 0::2] = q & 0xF
    out[:, 1::2] = q >> 4
    return out


def test_e8m0_is_a_bare_exponent():
    assert oracle.e8m0_decode(127) == 1.0 and oracle.e8m0_decode(128) == 2.0 and oracle.e8m0_decode(126) == 0.5
    assert oracle.e8m0_decode(0) == 2.0 ** -127 and oracle.e8m0_decode(254) == 2.0 ** 127
    for b in range(1, 255):
        assert oracle.e8m0_decode(b) == 2 * oracle.e8m0_decode(b - 1)


def test_scale_rule_cases():
    # shared exponent = floor(log2 amax) - 2: amax 6 -> 2^0; 4 -> 2^0; 3.99 -> 2^-1; 8 -> 2^1; 7.5 -> 2^0 (saturates)
    def scale_of(a):
        x = np.zeros((1, 32))
        x[0, 5] = a
        _, sf = oracle.mxfp4_quantize(bits(x))
        return int(sf[0, 0]) - 127
    assert scale_of(6.0) == 0 and scale_of(4.0) == 0 and scale_of(3.984375) == -1 and scale_of(8.0) == 1
    assert scale_of(7.5) == 0 and scale_of(1.0) == -2 and scale_of(2.0 ** -20) == -22 and scale_of(-96.0) == 4
    x = np.zeros((1, 32)); x[0, 0] = 7.5; x[0, 1] = -5.0; x[0, 2] = 0.25
    q, sf = oracle.mxfp4_quantize(bits(x))
    assert sf[0, 0] == 127 and list(nibbles(q)[0, :3]) == [7, 0xE, 0]      # 7.5 -> 6 (saturated), -5 -> -4 (tie to even), .25 -> 0


def test_hand_worked_block():
    # amax = 12 -> floor(log2 12) = 3 -> scale 2^1; x / 2 = [6, 3, 1.5, -0.75, 0.25, 2.5, -6, 0.05, 1.25, 0...]
    x = np.zeros((1, 32))
    x[0, :9] = [12, 6, 3, -1.5, 0.5, 5, -12, 0.1015625, 2.5]
    q, sf = oracle.mxfp4_quantize(bits(x))
    assert sf[0, 0] == 128
    assert list(nibbles(q)[0, :9]) == [7, 5, 3, 0xA, 0, 4, 0xF, 0, 2]      # -0.75 -> -1 (tie to even), 2.5 -> 2, 1.25 -> 1
    assert np.all(nibbles(q)[0, 9:] == 0)
    deq = oracle.mxfp4_dequantize(q, sf)
    assert list(deq[0, :9]) == [12, 6, 3, -2, 0, 4, -12, 0, 2]


def test_zero_block_signed_zero_and_extremes():
    x = np.zeros((1, 64))
    xb = bits(x)
    xb[0, 3] = 0x8000                       # -0
    q, sf = oracle.mxfp4_quantize(xb)
    assert sf[0, 0] == 0 and sf[0, 1] == 0 and nibbles(q)[0, 3] == 8 and np.count_nonzero(nibbles(q)[0] & 7) == 0
    big = np.zeros((1, 32), np.uint16)
    big[0, 0] = 0x7F7F                      # largest finite BF16, exponent 127 -> scale 2^125
    q, sf = oracle.mxfp4_quantize(big)
    assert sf[0, 0] == 252 and nibbles(q)[0, 0] == 7
    tiny = np.zeros((1, 32), np.uint16)
    tiny[0, 0] = 0x0001                     # smallest subnormal: the exponent clamps at -127
    q, sf = oracle.mxfp4_quantize(tiny)
    assert sf[0, 0] == 0 and nibbles(q)[0, 0] == 0


def test_exact_round_trip_of_grid_values_at_every_scale():
    vals = np.array([g for g in GRID] + [-g for g in GRID] + [6.0] * 16)
    for e in range(-120, 121, 7):
        xb = bits((vals * 2.0 ** e)[None, :])
        q, sf = oracle.mxfp4_quantize(xb)
        assert sf[0, 0] == e + 127
        assert np.array_equal(oracle.mxfp4_dequantize(q, sf)[0], vals * 2.0 ** e)


def test_against_exact_rational_definition():
    # independent restatement in rationals: S = 2^(floor(log2 amax) - 2), code = nearest grid point of x / S
    # (ties to the even code, saturating at 6)
    rng = np.random.default_rng(4)
    xb = rand_bits(rng, (6, 96), 3.0)
    q, sf = oracle.mxfp4_quantize(xb)
    x = oracle.bits_to_f64(xb)
    codes = nibbles(q)
    for r in range(6):
        for b in range(3):
            blk = [Fraction(v) for v in x[r, b * 32:(b + 1) * 32]]
            amax = max(abs(v) for v in blk)
            e = 0
            while Fraction(2) ** (e + 1) <= amax:
                e += 1
            while Fraction(2) ** e > amax:
                e -= 1
            S = Fraction(2) ** (e - 2)
            assert sf[r, b] == e - 2 + 127
            for k, v in enumerate(blk):
                y = abs(v) / S
                best = min(range(8), key=lambda c: (abs(Fraction(GRID[c]) - y), c & 1))
                if y >= 6:
                    best = 7
                want = best | (8 if v < 0 else 0)
                assert codes[r, b * 32 + k] == want


def test_invariants():
    rng = np.random.default_rng(5)
    xb = rand_bits(rng, (4, 128))
    q, sf = oracle.mxfp4_quantize(xb)
    qn, sfn = oracle.mxfp4_quantize(xb ^ 0x8000)
    assert np.array_equal(sfn, sf) and np.array_equal(nibbles(qn), nibbles(q) ^ 8)
    x8 = oracle.round_bf16(oracle.bits_to_f64(xb) * 8.0)
    q8, sf8 = oracle.mxfp4_quantize(x8)
    assert np.array_equal(q8, q) and np.array_equal(sf8, sf + 3)
    deq = oracle.mxfp4_dequantize(q, sf)
    x = oracle.bits_to_f64(xb)
    S = np.repeat(np.array([[oracle.e8m0_decode(b) for b in row] for row in sf]), 32, axis=1)
    sat = np.abs(x) > 6 * S
    assert np.all(np.abs(deq - x)[~sat] <= 1.0 * S[~sat]) and np.all(np.abs(deq[sat]) == 6 * S[sat])


def test_scale_storage_is_a_bijection_with_zero_padding():
    rows, K = 130, 288                      # 9 blocks per row: chunks of 4, last chunk padded
    sf = (np.arange(rows * 9).reshape(rows, 9) % 251 + 1).astype(np.uint8)
    sw = oracle.mx_sf_swizzle(sf, K)
    assert sw.size == 2 * 3 * 512
    offs = {oracle.mx_sf_swizzled_offset(r, b, K) for r in range(rows) for b in range(9)}
    assert len(offs) == rows * 9
    for r in (0, 31, 32, 127, 128, 129):
        for b in range(9):
            assert sw[oracle.mx_sf_swizzled_offset(r, b, K)] == sf[r, b]
    mask = np.ones(sw.size, bool)
    mask[list(offs)] = False
    assert np.all(sw[mask] == 0)
    assert oracle.mx_sf_swizzled_offset(33, 5, K) == 1 * 512 + 1 * 16 + 1 * 4 + 1


def test_linear_integer_exact_and_structure():
    rng = np.random.default_rng(6)
    M, N, K = 5, 7, 64
    qx = rng.integers(0, 256, size=(M, K // 2), dtype=np.uint8)
    qw = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    ex = rng.integers(-3, 4, size=(M, K // 32))
    ew = rng.integers(-3, 4, size=(N, K // 32))
    Y = oracle.mxfp4_linear(qx, (ex + 127).astype(np.uint8), qw, (ew + 127).astype(np.uint8))
    tw = [0, 1, 2, 3, 4, 6, 8, 12]
    val = lambda c: -tw[c & 7] if c & 8 else tw[c & 7]
    cx, cw = nibbles(qx), nibbles(qw)
    for m in range(M):
        for n in range(N):
            acc = Fraction(0)
            for k in range(K):
                acc += Fraction(val(cx[m, k]) * val(cw[n, k]), 4) * Fraction(2) ** int(ex[m, k // 32] + ew[n, k // 32])
            assert Fraction(Y[m, n]) == acc
    # bias and zero input
    bias = bits(np.arange(N) * 0.5)
    Y0 = oracle.mxfp4_linear(np.zeros_like(qx), (ex + 127).astype(np.uint8), qw, (ew + 127).astype(np.uint8), bias)
    assert np.array_equal(Y0, np.tile(np.arange(N) * 0.5, (M, 1)))
    # against a library matmul on the dequantized operands
    A = oracle.mxfp4_dequantize(qx, (ex + 127).astype(np.uint8))
    Bm = oracle.mxfp4_dequantize(qw, (ew + 127).astype(np.uint8))
    assert np.allclose(Y, A @ Bm.T, rtol=1e-13, atol=0)


def test_linear_quantized_is_linear_then_round_then_quantizer():
    # the composition the fused GPU epilogue is checked against: every step is one the tests above pin
    rng = np.random.default_rng(17)
    M, N, K = 6, 64, 64
    qx = rng.integers(0, 256, size=(M, K // 2), dtype=np.uint8)
    qw = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    sfx = (rng.integers(-1, 2, size=(M, K // 32)) + 127).astype(np.uint8)
    sfw = (rng.integers(-1, 2, size=(N, K // 32)) + 127).astype(np.uint8)
    H, h, q, sf = oracle.mxfp4_linear_quantized(qx, sfx, qw, sfw, None, oracle.ACT_NONE)
    Y = oracle.mxfp4_linear(qx, sfx, qw, sfw)
    assert np.array_equal(H, Y) and np.array_equal(h, oracle.round_bf16(Y))
    q2, sf2 = oracle.mxfp4_quantize(h)
    assert np.array_equal(q, q2) and np.array_equal(sf, sf2)
    # with the activation the pre-quantizer values are GELU of the linear
    Hg, hg, _, _ = oracle.mxfp4_linear_quantized(qx, sfx, qw, sfw, None, oracle.ACT_GELU_TANH)
    assert np.array_equal(Hg, oracle.gelu_tanh(Y)) and np.array_equal(hg, oracle.round_bf16(oracle.gelu_tanh(Y)))
    # dequantizing recovers every h to within the block's widest half step (1 unit) or its saturation distance
    deq = oracle.mxfp4_dequantize(q, sf)
    unit = np.repeat(np.ldexp(1.0, sf.astype(np.int32) - 127), 32, axis=1)
    hv = oracle.bits_to_f64(h)
    assert np.all(np.abs(deq - hv) <= np.maximum(unit, np.abs(hv) - 6 * unit) + 1e-12)
