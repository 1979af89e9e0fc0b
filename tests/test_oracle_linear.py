"""Pins for the oracle's matmuls -- CPU only.

Integer-exact brute force on tiny shapes (twice an E2M1 value is an integer and
power-of-two scales keep every product an integer multiple of a known power of
two), structural special cases, and a library matmul on exactly representable
inputs.
"""
import numpy as np
import torch

import oracle

TWICE = [0, 1, 2, 3, 4, 6, 8, 12]  # 2 * E2M1 magnitude, by code


def twice_value(code: int) -> int:
    return -TWICE[code & 7] if code & 8 else TWICE[code & 7]


def random_quantized(rng, rows, K, exps=(-2, 3)):
    """Random nibbles and power-of-two E4M3 scales (normal codes with zero mantissa)."""
    q = rng.integers(0, 256, size=(rows, K // 2), dtype=np.uint8)
    e = rng.integers(exps[0], exps[1] + 1, size=(rows, K // 16))
    sf = ((e + 7) << 3).astype(np.uint8)
    return q, sf, e


def int_matmul(qx, ex, qw, ew, shift):
    """sum_k (2qx)(2qw) 2^(ex+ew+shift) in Python integers (exact)."""
    M, N, K = qx.shape[0], qw.shape[0], qx.shape[1] * 2
    out = [[0] * N for _ in range(M)]
    for m in range(M):
        for n in range(N):
            acc = 0
            for k in range(K):
                cx = (int(qx[m, k // 2]) >> (4 * (k & 1))) & 0xF
                cw = (int(qw[n, k // 2]) >> (4 * (k & 1))) & 0xF
                acc += twice_value(cx) * twice_value(cw) << (int(ex[m, k // 16]) + int(ew[n, k // 16]) + shift)
            out[m][n] = acc
    return out


def test_tiny_nvfp4_matmul_equals_integer_brute_force():
    rng = np.random.default_rng(0)
    for (M, N, K) in [(3, 5, 16), (8, 8, 32), (4, 7, 64), (2, 3, 128)]:
        qx, sfx, ex = random_quantized(rng, M, K)
        qw, sfw, ew = random_quantized(rng, N, K)
        Y = oracle.nvfp4_linear(qx, sfx, 1.0, qw, sfw, 1.0)
        want = int_matmul(qx, ex, qw, ew, shift=4)  # scales >= 2^-2 each -> shift 4 keeps integers
        for m in range(M):
            for n in range(N):
                # Y * 4 (two halvings) * 2^4 == integer sum
                assert Y[m, n] * 4 * 16 == want[m][n]


def test_tensor_scales_and_bias_enter_linearly():
    rng = np.random.default_rng(1)
    qx, sfx, _ = random_quantized(rng, 4, 64)
    qw, sfw, _ = random_quantized(rng, 6, 64)
    Y1 = oracle.nvfp4_linear(qx, sfx, 1.0, qw, sfw, 1.0)
    Y2 = oracle.nvfp4_linear(qx, sfx, 0.25, qw, sfw, 8.0)
    assert np.array_equal(Y2, Y1 * 2.0)
    bias = torch.tensor([0.5, -1.0, 2.0, 0.0, 3.0, -0.25]).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    Yb = oracle.nvfp4_linear(qx, sfx, 1.0, qw, sfw, 1.0, bias)
    assert np.array_equal(Yb - Y1, np.tile([0.5, -1.0, 2.0, 0.0, 3.0, -0.25], (4, 1)))


def test_zero_activations_give_bias_and_identity_weight_gives_dequantized_input():
    rng = np.random.default_rng(2)
    K = 32
    qx, sfx, _ = random_quantized(rng, 5, K)
    # W = 2 * I: each row n has code(+1.0)=2 at column n, scale 2.0 in that column's block
    qw = np.zeros((K, K // 2), np.uint8)
    sfw = np.zeros((K, K // 16), np.uint8)
    for n in range(K):
        qw[n, n // 2] = 2 << (4 * (n & 1))
        sfw[n, n // 16] = (1 + 7) << 3
    Y = oracle.nvfp4_linear(qx, sfx, 1.0, qw, sfw, 1.0)
    assert np.array_equal(Y, 2.0 * oracle.dequantize(qx, sfx, 1.0))
    bias = np.full(K, 0x3FC0, np.uint16)  # 1.5
    Y0 = oracle.nvfp4_linear(np.zeros_like(qx), sfx, 1.0, qw, sfw, 1.0, bias)
    assert np.all(Y0 == 1.5)


def test_k_split_additivity_and_row_selection():
    rng = np.random.default_rng(3)
    qx, sfx, _ = random_quantized(rng, 9, 128)
    qw, sfw, _ = random_quantized(rng, 4, 128)
    Y = oracle.nvfp4_linear(qx, sfx, 1.0, qw, sfw, 1.0)
    Ya = oracle.nvfp4_linear(qx[:, :32], sfx[:, :4], 1.0, qw[:, :32], sfw[:, :4], 1.0)
    Yb = oracle.nvfp4_linear(qx[:, 32:], sfx[:, 4:], 1.0, qw[:, 32:], sfw[:, 4:], 1.0)
    assert np.array_equal(Y, Ya + Yb)  # all partial sums are exact here
    rows = [7, 0, 3]
    assert np.array_equal(oracle.nvfp4_linear(qx, sfx, 1.0, qw, sfw, 1.0, rows=rows), Y[rows])


def test_transposed_operand_or_wrong_nibble_order_would_be_caught():
    # one non-zero element in X and in W at different positions inside one byte
    K = 16
    qx = np.zeros((1, K // 2), np.uint8)
    qw = np.zeros((2, K // 2), np.uint8)
    sf = np.full((1, 1), 0x38, np.uint8)
    qx[0, 1] = 0x20            # element k=3 (high nibble of byte 1) = +1.0
    qw[0, 1] = 0x40            # row 0: k=3 = +2.0
    qw[1, 1] = 0x04            # row 1: k=2 = +2.0
    Y = oracle.nvfp4_linear(qx, sf, 1.0, qw, np.repeat(sf, 2, 0), 1.0)
    assert Y.tolist() == [[2.0, 0.0]]


def test_bf16_linear_against_integer_matmul_and_library():
    rng = np.random.default_rng(4)
    M, N, K = 7, 5, 48
    xi = rng.integers(-8, 9, size=(M, K))
    wi = rng.integers(-8, 9, size=(N, K))
    bi = rng.integers(-4, 5, size=(N,))
    tb = lambda a: torch.tensor(a, dtype=torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    Y = oracle.bf16_linear(tb(xi), tb(wi), tb(bi))
    assert np.array_equal(Y, (xi @ wi.T + bi).astype(np.float64))
    # general BF16 values against numpy's FP64 matmul (a library routine on exact inputs)
    x = torch.randn(M, K, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    w = torch.randn(N, K, generator=torch.Generator().manual_seed(2)).to(torch.bfloat16)
    Y = oracle.bf16_linear(x.view(torch.int16).numpy().view(np.uint16), w.view(torch.int16).numpy().view(np.uint16))
    ref = x.double().numpy() @ w.double().numpy().T
    assert np.allclose(Y, ref, rtol=1e-13, atol=1e-13)
    assert np.array_equal(oracle.bf16_linear(tb(xi), tb(wi), rows=[2, 6]), (xi @ wi.T)[[2, 6]].astype(np.float64))


def test_linear_tolerance_formula():
    Y = np.array([[3.0, -4.0], [0.0, 0.0]])
    tol = oracle.linear_tolerance(Y)
    rms0 = np.sqrt((9 + 16) / 2)
    assert np.allclose(tol[0], [3 / 128 + 1e-4 * rms0, 4 / 128 + 1e-4 * rms0])
    assert np.all(tol[1] == 0)
