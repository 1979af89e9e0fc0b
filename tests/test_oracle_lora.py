"""Pins for the oracle's adapter merge (weight refresh) -- CPU only.

None of these re-types the oracle's loop: exact integer arithmetic, an FP64 library product,
two cases worked by hand whose answers depend on the order of the binary32 sum and on the single
rounding of the last multiply-add, and structural special cases.
"""
from fractions import Fraction

import numpy as np
import torch

import oracle


def bits(values) -> np.ndarray:
    """Exactly representable values -> BF16 bit patterns (asserts nothing is rounded)."""
    t = torch.tensor(np.asarray(values, dtype=np.float64), dtype=torch.float64)
    h = t.to(torch.bfloat16)
    assert torch.equal(h.to(torch.float64), t), "test input not representable in BF16"
    return h.view(torch.int16).numpy().view(np.uint16)


def rand_bits(rng, shape, scale=1.0) -> np.ndarray:
    t = torch.from_numpy(rng.standard_normal(shape) * scale).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def test_integer_exact_against_integer_arithmetic():
    # small integers: every product, partial sum and result is an integer below 2^8, so
    # binary32 and BF16 hold them exactly and the merge must equal integer arithmetic
    rng = np.random.default_rng(11)
    N, K, r = 24, 48, 32
    W = rng.integers(-40, 41, size=(N, K))
    A = rng.integers(-1, 2, size=(r, K))
    B = rng.integers(-1, 2, size=(N, r))
    s = 2
    want = W + s * (B @ A)
    assert np.abs(want).max() <= 256 and np.abs(B @ A).max() <= 64
    got = oracle.bits_to_f64(oracle.lora_merge(bits(W), bits(A), bits(B), float(s)))
    assert np.array_equal(got, want.astype(np.float64))


def test_not_transposed_and_rank_index():
    # one non-zero entry in each factor: B[n0, j0] * A[j0, k0] lands on W'[n0, k0] only
    N, K, r = 5, 32, 4
    W = np.zeros((N, K))
    for (n0, j0, k0) in [(0, 0, 0), (3, 2, 17), (4, 3, 31)]:
        A = np.zeros((r, K))
        B = np.zeros((N, r))
        A[j0, k0] = 3.0
        B[n0, j0] = 0.5
        got = oracle.bits_to_f64(oracle.lora_merge(bits(W), bits(A), bits(B), 2.0))
        want = np.zeros((N, K))
        want[n0, k0] = 3.0
        assert np.array_equal(got, want)


def test_zero_adapter_returns_base_weights():
    rng = np.random.default_rng(5)
    Wb = rand_bits(rng, (16, 64), 0.02)
    Wb[Wb == 0x8000] = 0  # a negative zero would come back as +0 (0 * s + -0 = +0)
    Ab = rand_bits(rng, (32, 64))
    Zb = np.zeros((16, 32), np.uint16)
    assert np.array_equal(oracle.lora_merge(Wb, Ab, Zb, 2.0), Wb)
    assert np.array_equal(oracle.lora_merge(Wb, np.zeros((32, 64), np.uint16), rand_bits(rng, (16, 32)), 2.0), Wb)


def test_order_of_the_binary32_sum_by_hand():
    # products 2^24, 1, -2^24 in this order: 2^24 + 1 rounds back to 2^24 (tie to even), so the
    # running sum ends at 0 and W' = W; any other order (or a wider accumulator) gives W + 2
    A = np.array([[4096.0], [1.0], [4096.0]])          # [r=3, K=1]
    B = np.array([[4096.0, 1.0, -4096.0]])             # [N=1, r=3]
    W = np.array([[0.5]])
    Ab = np.zeros((3, 16), np.uint16)
    Ab[:, :1] = bits(A)
    Wb = np.zeros((1, 16), np.uint16)
    Wb[:, :1] = bits(W)
    out = oracle.bits_to_f64(oracle.lora_merge(Wb, Ab, bits(B), 2.0))
    assert out[0, 0] == 0.5
    # reversed rank order: -2^24 + 1 = -16777215 is exact, + 2^24 = 1  ->  W' = 0.5 + 2 = 2.5
    out = oracle.bits_to_f64(oracle.lora_merge(Wb, Ab[::-1].copy(), bits(B[:, ::-1].copy()), 2.0))
    assert out[0, 0] == 2.5


def test_last_multiply_add_rounds_once_by_hand():
    # acc = 1 + 2^-23 (exact), s = 3, w = -3: the fused result is 3 * 2^-23 exactly.  Rounding
    # the product first would give 3 + 2^-21 (tie to even) and then 2^-21 = 4 * 2^-23.
    A = np.array([[1.0], [2.0 ** -12]])
    B = np.array([[1.0, 2.0 ** -11]])
    Ab = np.zeros((2, 16), np.uint16)
    Ab[:, :1] = bits(A)
    Wb = np.zeros((1, 16), np.uint16)
    Wb[:, :1] = bits([[-3.0]])
    out = oracle.bits_to_f64(oracle.lora_merge(Wb, Ab, bits(B), 3.0))
    assert out[0, 0] == 3.0 * 2.0 ** -23
    # the same through exact rationals: one rounding of s*acc + w, then one to BF16
    exact = Fraction(3) * (1 + Fraction(1, 2 ** 23)) - 3
    assert Fraction(out[0, 0]) == exact


def test_agrees_with_fp64_library_product_to_the_last_place():
    # W + s * (B @ A) in FP64 (numpy's matmul), rounded once to BF16: the binary32 chain may
    # differ only where the exact value sits next to a BF16 rounding boundary, and then by one
    # unit in the last place
    rng = np.random.default_rng(2)
    N, K, r = 96, 160, 32
    Wb = rand_bits(rng, (N, K), K ** -0.5)
    Ab = rand_bits(rng, (r, K), 0.05)
    Bb = rand_bits(rng, (N, r), 0.05)
    W, A, B = (oracle.bits_to_f64(x) for x in (Wb, Ab, Bb))
    want_bits = oracle.round_bf16(W + 2.0 * (B @ A))
    got_bits = oracle.lora_merge(Wb, Ab, Bb, 2.0)
    differ = got_bits != want_bits
    assert differ.mean() < 0.01
    # neighbouring BF16 values of one sign have neighbouring bit patterns
    d = np.abs(got_bits.astype(np.int64) - want_bits.astype(np.int64))
    assert d.max() <= 1
    # and the adapter is really in there: dropping it changes a large share of the weights
    assert (oracle.round_bf16(W) != got_bits).mean() > 0.5


def test_scaling_is_linear_in_powers_of_two():
    # with s a power of two, s*(B A) only shifts exponents: merge(W, A, B, 4) == merge(W, A, 4B, 1)
    rng = np.random.default_rng(8)
    Wb = rand_bits(rng, (8, 32), 0.1)
    Ab = rand_bits(rng, (16, 32), 0.1)
    Bb = rand_bits(rng, (8, 16), 0.1)
    B4 = oracle.round_bf16(4.0 * oracle.bits_to_f64(Bb))
    assert np.array_equal(oracle.lora_merge(Wb, Ab, Bb, 4.0), oracle.lora_merge(Wb, Ab, B4, 1.0))


def test_requantize_is_merge_then_weight_quantizer():
    rng = np.random.default_rng(4)
    Wb = rand_bits(rng, (32, 64), 0.05)
    Ab = rand_bits(rng, (32, 64), 0.05)
    Bb = rand_bits(rng, (32, 32), 0.05)
    merged, q, sf, T = oracle.requantize_lora(Wb, Ab, Bb, 2.0)
    amax = np.abs(oracle.bits_to_f64(merged)).max()
    assert T == np.float32(np.float32(amax) / np.float32(2688.0))
    # dequantized merged weights stay within half an FP4 step of the block scale times T
    deq = oracle.dequantize(q, sf, T)
    step = np.repeat(np.array([oracle.e4m3_decode(int(c)) for c in sf.ravel()]).reshape(sf.shape), 16, axis=1) * float(T)
    err = np.abs(deq - oracle.bits_to_f64(merged))
    assert np.all(err <= 1.0 * step + 1e-30)  # widest E2M1 gap is 2 (between 4 and 6): half of it is 1
