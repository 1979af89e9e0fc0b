"""Pins for the oracle's NVFP4 quantizer -- CPU only.

Hand-worked block (tests/golden), block-scale cases, exact round trips, the
exact-rational model on random blocks, metamorphic invariants, the error bound,
and the scale-storage index map.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import exact
from paper_2604_06916_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "nvfp4_block_example.txt")


def bits(values) -> np.ndarray:
    t = torch.tensor(values, dtype=torch.float32).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def codes_of(q_row: np.ndarray) -> list[int]:
    out = []
    for b in q_row:
        out += [int(b) & 0xF, int(b) >> 4]
    return out


def read_golden():
    fields = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split("=")
        fields[k.strip()] = v.split()
    return fields


def test_hand_worked_block_from_golden_file():
    g = read_golden()
    x = bits([[float(v) for v in g["x"]]])
    q, sf = oracle.quantize(x, float(g["T"][0]))
    assert int(sf[0, 0]) == int(g["scale"][0], 16)
    assert codes_of(q[0]) == [int(c) for c in g["codes"]]
    assert [int(b) for b in q[0]] == [int(b, 16) for b in g["bytes"]]


@pytest.mark.parametrize("amax,scale_byte,top_code,top_deq", [
    (6.0, 0x38, 7, 6.0),
    (6.25, 0x38, 7, 6.0),     # 6.25/6 = 1.0417 < 1.0625 -> scale 1.0, the max saturates at 6*scale
    (6.5, 0x39, 7, 6.75),     # 1.0833 -> 1.125; 6.5/1.125 = 5.78 -> 6
    (6.375, 0x38, 7, 6.0),    # 1.0625 is an exact tie -> even mantissa -> 1.0
    (3.0, 0x30, 7, 3.0),
])
def test_block_scale_is_amax_over_6_rounded_to_e4m3(amax, scale_byte, top_code, top_deq):
    x = bits([[amax] + [0.0] * 15])
    q, sf = oracle.quantize(x, 1.0)
    assert int(sf[0, 0]) == scale_byte
    assert codes_of(q[0])[0] == top_code
    assert oracle.dequantize(q, sf, 1.0)[0, 0] == top_deq


def test_zero_block_and_zero_tensor():
    x = bits([[0.0, -0.0] * 8 + [1.0] * 16])
    assert oracle.tensor_scale(bits([[0.0] * 16])) == np.float32(1.0)
    q, sf = oracle.quantize(x, 1.0)
    assert int(sf[0, 0]) == 0
    assert codes_of(q[0])[:16] == [0, 8] * 8  # magnitudes 0, sign bits kept
    assert np.all(oracle.dequantize(q, sf, 1.0)[0, :16] == 0.0)


def test_tensor_scale_definition():
    x = bits([[1.0, -2688.0, 3.0, 0.5] * 4])
    assert oracle.tensor_scale(x) == np.float32(1.0)
    x = bits([[0.75] * 16])
    assert oracle.tensor_scale(x) == np.float32(0.75) / np.float32(2688.0)


@pytest.mark.parametrize("T", [1.0, 2.0 ** -3])
def test_exact_round_trip_of_grid_values(T):
    grid = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    signed = grid + [-g for g in grid[1:]] + [6.0]  # 16 entries, max magnitude 6
    for code in range(0x08, 0x7F):  # normal E4M3 scales
        s = oracle.e4m3_decode(code)
        if s * T * 0.5 < 2.0 ** -126 or s * T * 6 > 3e38:
            continue
        vals = [g * s * T for g in signed]
        x = bits([vals])
        assert np.array_equal(oracle.bits_to_f64(x)[0], np.array(vals))  # representable in BF16
        q, sf = oracle.quantize(x, T)
        assert int(sf[0, 0]) == code
        assert np.array_equal(oracle.dequantize(q, sf, T)[0], np.array(vals))


def _random_blocks(seed, n, kind):
    gen = torch.Generator().manual_seed(seed)
    return workloads.to_bits(workloads.make_activation(kind, n, 16, gen, "cpu"))


@pytest.mark.parametrize("kind", ["outlier", "student_t", "channel"])
def test_rounded_rational_model_matches_c_oracle_bit_for_bit(kind):
    x = _random_blocks(5, 300, kind)
    for T in (np.float32(1.0), oracle.tensor_scale(x)):
        q, sf = oracle.quantize(x, T)
        for r in range(x.shape[0]):
            sb, codes = exact.quantize_block_rounded([int(h) for h in x[r]], Fraction(float(T)))
            assert sb == int(sf[r, 0])
            assert codes == codes_of(q[r])


def test_exact_division_model_differs_rarely_and_only_by_adjacent_codes():
    x = _random_blocks(9, 400, "student_t")
    T = np.float32(2.0 ** -2)  # power of two: scale step must agree exactly
    q, sf = oracle.quantize(x, T)
    diff = total = 0
    for r in range(x.shape[0]):
        sb, codes = exact.quantize_block_exact([int(h) for h in x[r]], Fraction(float(T)))
        assert sb == int(sf[r, 0])
        for a, b in zip(codes, codes_of(q[r])):
            total += 1
            if a != b:
                diff += 1
                assert (a & 8) == (b & 8) and abs((a & 7) - (b & 7)) == 1
    assert diff <= max(1, total // 2000)


def test_metamorphic_negation_scaling_permutation():
    x = _random_blocks(21, 64, "outlier").reshape(16, 64)
    T = oracle.tensor_scale(x)
    q, sf = oracle.quantize(x, T)
    qn, sfn = oracle.quantize(x ^ np.uint16(0x8000), T)
    assert np.array_equal(sfn, sf) and np.array_equal(qn, q ^ np.uint8(0x88))
    x4 = (oracle.bits_to_f64(x) * 4.0).astype(np.float32)
    x4b = torch.from_numpy(x4).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    q4, sf4 = oracle.quantize(x4b, np.float32(T * 4))
    assert np.array_equal(q4, q) and np.array_equal(sf4, sf)
    perm = np.random.default_rng(0).permutation(x.shape[0])
    qp, sfp = oracle.quantize(x[perm], T)
    assert np.array_equal(qp, q[perm]) and np.array_equal(sfp, sf[perm])


def test_error_bound_and_range():
    x = _random_blocks(33, 2048, "student_t").reshape(256, 128)
    T = oracle.tensor_scale(x)
    q, sf = oracle.quantize(x, T)
    xr = oracle.bits_to_f64(x)
    xh = oracle.dequantize(q, sf, T)
    assert np.max(np.abs(xh)) <= 6 * 448 * float(T) * (1 + 1e-12)
    s = np.repeat(np.array([[oracle.e4m3_decode(int(b)) for b in row] for row in sf]), 16, axis=1) * float(T)
    mag = np.abs(xh) / np.where(s == 0, 1, s)
    step = np.select([mag < 2, mag < 4], [0.5, 1.0], 2.0)  # local grid spacing
    inside = (np.abs(xr) <= 6 * s) & (s > 0)
    err = np.abs(xr - xh)
    assert np.all(err[inside] <= (step[inside] / 2) * s[inside] * (1 + 1e-6))
    # saturated elements land on +-6*s
    sat = (np.abs(xr) > 6 * s) & (s > 0)
    assert np.all(np.abs(xh[sat]) == 6 * s[sat])


def test_scale_storage_map_is_a_bijection_with_zero_padding():
    for rows, K in [(128, 64), (130, 160), (257, 2240), (40, 5600)]:
        nb = K // 16
        total = oracle.sf_swizzled_bytes(rows, K)
        assert total == -(-rows // 128) * -(-nb // 4) * 512
        offs = {oracle.sf_swizzled_offset(r, b, K) for r in range(rows) for b in range(nb)}
        assert len(offs) == rows * nb and max(offs) < total and min(offs) >= 0
        sf = (np.arange(rows * nb, dtype=np.int64) % 251 + 1).astype(np.uint8).reshape(rows, nb)
        sw = oracle.sf_swizzle(sf, K)
        assert int(np.count_nonzero(sw)) == rows * nb
        for r, b in [(0, 0), (rows - 1, nb - 1), (rows // 2, nb // 3), (min(rows - 1, 37), 1)]:
            assert sw[oracle.sf_swizzled_offset(r, b, K)] == sf[r, b]
    # the formula inside one 512-byte chunk: 32 lines of 16 bytes, 4 row groups x 4 blocks per line
    assert oracle.sf_swizzled_offset(0, 1, 64) == 1
    assert oracle.sf_swizzled_offset(1, 0, 64) == 16
    assert oracle.sf_swizzled_offset(32, 0, 64) == 4
    assert oracle.sf_swizzled_offset(127, 3, 64) == 31 * 16 + 3 * 4 + 3
    assert oracle.sf_swizzled_offset(0, 4, 128) == 512
    assert oracle.sf_swizzled_offset(128, 0, 128) == 1024
