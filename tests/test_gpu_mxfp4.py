"""GPU parity: MXFP4 quantizer (bit-exact) and linear (tolerance / integer-exact) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_06916_b200 import workloads
from tests.helpers import bits_of, check_linear, from_bits, sample_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06916_b200 import binding
    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def mx_offsets(rows, K):
    nb = K // 32
    chunks_k = (nb + 3) // 4
    r = np.asarray(rows, dtype=np.int64)[:, None]
    b = np.arange(nb, dtype=np.int64)[None, :]
    rr = r % 128
    return ((r // 128) * chunks_k + b // 4) * 512 + (rr % 32) * 16 + (rr // 32) * 4 + b % 4


def test_offset_helper_matches_oracle_rule():
    K = 416
    offs = mx_offsets(np.array([0, 31, 32, 127, 128, 300]), K)
    for i, r in enumerate([0, 31, 32, 127, 128, 300]):
        for b in range(K // 32):
            assert offs[i, b] == oracle.mx_sf_swizzled_offset(r, b, K)


@pytest.mark.parametrize("M,K,pad", [(256, 512, 0), (1, 32, 0), (130, 160, 0), (257, 2240, 8), (40, 5600, 64), (300, 96, 32)])
def test_quantizer_bit_exact_both_layouts(B, M, K, pad):
    g = torch.Generator(device="cuda").manual_seed(M + K)
    big = workloads.make_activation("outlier", M, K + pad, g, "cuda") * 3.0
    x = big[:, :K]
    xb = bits_of(x.contiguous())
    want_q, want_sf = oracle.mxfp4_quantize(xb)
    q, sf = B.mxfp4_quantize(x, B.SF_ROW_MAJOR)
    assert np.array_equal(q.cpu().numpy(), want_q)
    assert np.array_equal(sf.cpu().numpy().reshape(M, K // 32), want_sf)
    q2, sf2 = B.mxfp4_quantize(x, B.SF_SWIZZLED_128x4)
    assert np.array_equal(q2.cpu().numpy(), want_q)
    assert np.array_equal(sf2.cpu().numpy(), oracle.mx_sf_swizzle(want_sf, K))      # padding bytes are 0


def test_quantizer_special_values(B):
    vals = np.zeros((2, 64))
    vals[0, :9] = [12, 6, 3, -1.5, 0.5, 5, -12, 0.1015625, 2.5]
    vals[1, :6] = [7.5, -5.0, 0.25, 2.0 ** -20, -2.0 ** -30, 1e-38]
    xb = bits_of(torch.tensor(vals, dtype=torch.float64).to(torch.bfloat16))
    xb[1, 40] = 0x8000     # -0
    xb[1, 41] = 0x0001     # smallest subnormal
    xb[0, 63] = 0x7F7F     # largest finite
    x = from_bits(xb, "cuda")
    q, sf = B.mxfp4_quantize(x, B.SF_ROW_MAJOR)
    want_q, want_sf = oracle.mxfp4_quantize(xb)
    assert np.array_equal(q.cpu().numpy(), want_q) and np.array_equal(sf.cpu().numpy().reshape(2, 2), want_sf)


@pytest.mark.parametrize("M,N,K", [(256, 256, 64), (128, 192, 256), (256, 384, 512), (130, 200, 96), (64, 8, 32),
                                   (300, 456, 448), (200, 264, 1312)])
def test_linear_integer_exact(B, M, N, K):
    rng = np.random.default_rng(M + N + K)
    qx = rng.integers(0, 256, size=(M, K // 2), dtype=np.uint8)
    qw = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    sfx = (rng.integers(-2, 3, size=(M, K // 32)) + 127).astype(np.uint8)
    sfw = (rng.integers(-2, 3, size=(N, K // 32)) + 127).astype(np.uint8)
    Y = oracle.mxfp4_linear(qx, sfx, qw, sfw)
    if np.abs(Y).max() * 4 >= 2 ** 24:
        pytest.skip("sum too large for an exact FP32 accumulator")
    y = B.mxfp4_linear(dev(qx), dev(oracle.mx_sf_swizzle(sfx, K)), dev(qw), dev(oracle.mx_sf_swizzle(sfw, K)))
    B.sol_last_device_status()
    got, want = bits_of(y), oracle.round_bf16(Y)
    bad = got != want
    assert not bad.any(), (f"{int(bad.sum())} of {bad.size} differ; rows {np.unique(np.argwhere(bad)[:, 0])[:10]} "
                           f"cols {np.unique(np.argwhere(bad)[:, 1])[:10]}")


def test_scale_placement_probe(B):
    # one non-zero row of X whose 32-element blocks carry distinct scales, against one-hot rows of W:
    # every output isolates one (row, block) scale and one nibble position
    M, N, K = 256, 256, 512
    for row in (0, 77, 128, 255):
        qx = np.zeros((M, K // 2), np.uint8)
        sfx = np.full((M, K // 32), 127, np.uint8)
        qx[row, :] = 0x22                                   # every element 1.0
        sfx[row, :] = (np.arange(K // 32) % 7 + 124).astype(np.uint8)
        qw = np.zeros((N, K // 2), np.uint8)
        sfw = np.full((N, K // 32), 127, np.uint8)
        ks = (np.arange(N) * 37 + 5) % K
        for n, k in enumerate(ks):
            qw[n, k // 2] = 0x2 << (4 * (k & 1))
            sfw[n, k // 32] = (n % 5) + 125
        Y = oracle.mxfp4_linear(qx, sfx, qw, sfw)
        y = B.mxfp4_linear(dev(qx), dev(oracle.mx_sf_swizzle(sfx, K)), dev(qw), dev(oracle.mx_sf_swizzle(sfw, K)))
        assert np.array_equal(bits_of(y), oracle.round_bf16(Y)), f"row {row}"
        assert np.count_nonzero(Y) == N


@pytest.mark.parametrize("index", [1, 5])   # FLUX d_proj and s_out at full size, sampled rows
def test_flux_layers_sampled_rows(B, index):
    cfg = workloads.CONFIG_FLUX
    layer = cfg.layers[index]
    X, W, bias = workloads.make_layer(cfg, index, "cuda")
    M, K, N = layer.M, layer.K, layer.N
    xq, xsf = B.mxfp4_quantize(X)
    wq, wsf = B.mxfp4_quantize(W)
    y = B.mxfp4_linear(xq, xsf, wq, wsf, bias)
    B.sol_last_device_status()
    rows = sample_rows(M, seed=index)
    rows_t = torch.from_numpy(rows).cuda()
    # quantizer outputs of the sampled rows and of W, bit for bit
    want_qx, want_sfx = oracle.mxfp4_quantize(bits_of(X[rows_t]))
    want_qw, want_sfw = oracle.mxfp4_quantize(bits_of(W))
    assert np.array_equal(xq[rows_t].cpu().numpy(), want_qx)
    assert np.array_equal(xsf.cpu().numpy()[mx_offsets(rows, K)], want_sfx)
    assert np.array_equal(wq.cpu().numpy(), want_qw)
    assert np.array_equal(wsf.cpu().numpy(), oracle.mx_sf_swizzle(want_sfw, K))
    Y = oracle.mxfp4_linear(want_qx, want_sfx, want_qw, want_sfw, bits_of(bias))
    check_linear(bits_of(y[rows_t]), Y, f"{cfg.name}/{layer.name} mxfp4")


@pytest.mark.parametrize("M,N,K", [(256, 256, 64), (128, 384, 256), (300, 512, 448), (64, 128, 32), (520, 1024, 512)])
def test_quantized_output_integer_exact_bit_for_bit(B, M, N, K):
    rng = np.random.default_rng(M * 5 + N + K)
    qx = rng.integers(0, 256, size=(M, K // 2), dtype=np.uint8)
    qw = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    sfx = (rng.integers(-2, 3, size=(M, K // 32)) + 127).astype(np.uint8)
    sfw = (rng.integers(-2, 3, size=(N, K // 32)) + 127).astype(np.uint8)
    H, h, q_star, sf_star = oracle.mxfp4_linear_quantized(qx, sfx, qw, sfw, None, oracle.ACT_NONE)
    if np.abs(H).max() * 4 >= 2 ** 24:
        pytest.skip("sum too large for an exact FP32 accumulator")
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    hq, hsf = B.mxfp4_linear_quantized_out(dev(qx), dev(oracle.mx_sf_swizzle(sfx, K)), dev(qw),
                                           dev(oracle.mx_sf_swizzle(sfw, K)), None, B.ACT_NONE, amax_out=amax)
    B.sol_last_device_status()
    assert np.array_equal(hq.cpu().numpy(), q_star)
    assert np.array_equal(hsf.cpu().numpy(), oracle.mx_sf_swizzle(sf_star, N))      # padding rows are 0
    assert amax.item() == np.abs(oracle.bits_to_f64(h)).max()


@pytest.mark.parametrize("M,N,K", [(384, 512, 1024), (1000, 384, 96), (4608, 1536, 3072)])
def test_quantized_output_equals_linear_then_quantizer(B, M, N, K):
    # without an activation the fused epilogue rounds the same FP32 accumulator to BF16 and applies the same
    # quantizer arithmetic as mxfp4_linear followed by mxfp4_quantize (both checked against the oracle above)
    g = torch.Generator(device="cuda").manual_seed(M + N + K)
    X = workloads.make_activation("student_t", M, K, g, "cuda")
    W = (torch.randn(N, K, generator=g, device="cuda") * K ** -0.5).to(torch.bfloat16)
    bias = (torch.randn(N, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    xq, xsf = B.mxfp4_quantize(X)
    wq, wsf = B.mxfp4_quantize(W)
    y = B.mxfp4_linear(xq, xsf, wq, wsf, bias)
    want_q, want_sf = B.mxfp4_quantize(y)
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    hq, hsf = B.mxfp4_linear_quantized_out(xq, xsf, wq, wsf, bias, B.ACT_NONE, amax_out=amax)
    B.sol_last_device_status()
    assert torch.equal(hq, want_q) and torch.equal(hsf, want_sf)
    assert amax.item() == y.float().abs().max().item()


def test_quantized_output_with_gelu_against_oracle(B):
    M, N, K = 300, 256, 512
    g = torch.Generator(device="cuda").manual_seed(99)
    X = workloads.make_activation("student_t", M, K, g, "cuda")
    W = (torch.randn(N, K, generator=g, device="cuda") * K ** -0.5).to(torch.bfloat16)
    bias = (torch.randn(N, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    qx, sfx = oracle.mxfp4_quantize(bits_of(X))
    qw, sfw = oracle.mxfp4_quantize(bits_of(W))
    H, h, q_star, sf_star = oracle.mxfp4_linear_quantized(qx, sfx, qw, sfw, bits_of(bias), oracle.ACT_GELU_TANH)
    hq, hsf = B.mxfp4_linear_quantized_out(dev(qx), dev(oracle.mx_sf_swizzle(sfx, K)), dev(qw),
                                           dev(oracle.mx_sf_swizzle(sfw, K)), bias, B.ACT_GELU_TANH)
    B.sol_last_device_status()
    sf_rm = hsf.cpu().numpy()[mx_offsets(np.arange(M), N)]
    # scale bytes: the block maximum may sit on either side of a power of two in a few blocks, never further
    d = np.abs(sf_rm.astype(np.int32) - sf_star.astype(np.int32))
    assert d.max() <= 1 and (d == 0).mean() >= 0.99
    # every dequantized value within the format's widest half step (1 unit of the emitted scale), or its
    # saturation distance, plus the linear's tolerance (GELU's slope is below 1.13) of the FP64 result
    deq = oracle.mxfp4_dequantize(hq.cpu().numpy(), sf_rm)
    scale = np.repeat(np.ldexp(1.0, sf_rm.astype(np.int32) - 127), 32, axis=1)
    Y = oracle.mxfp4_linear(qx, sfx, qw, sfw, bits_of(bias))
    tol = 1.2 * oracle.linear_tolerance(Y) + 2.0 ** -8 * np.abs(H)
    # (a block maximum up to 8 units saturates at the largest code, 6 units)
    reach = np.maximum(1.0 * scale, np.abs(H) - 6.0 * scale)
    assert np.all(np.abs(deq - H) <= reach * (1 + 2.0 ** -6) + tol)
    # and it is the oracle's own output almost everywhere
    assert (hq.cpu().numpy() == q_star).mean() >= 0.98


def pow2_mx(rng, rows, K):
    """Random nibbles with power-of-two MXFP4 scales in a narrow range: sums stay exact in FP32."""
    q = rng.integers(0, 256, size=(rows, K // 2), dtype=np.uint8)
    return q, (rng.integers(-2, 3, size=(rows, K // 32)) + 127).astype(np.uint8)


def concat_reference(B, parts):
    """MXFP4 of the column-wise concatenation of BF16 tensors, from the library's own quantizer (itself bit for
    bit the oracle's, see above)."""
    return B.mxfp4_quantize(torch.cat(parts, dim=1).contiguous())


@pytest.mark.parametrize("M,K1,K2", [(256, 128, 256), (300, 384, 128), (130, 1024, 3072)])
def test_quantize_into_two_slices_equals_quantizer_on_the_concatenation(B, M, K1, K2):
    g = torch.Generator(device="cuda").manual_seed(M + K1)
    a = workloads.make_activation("student_t", M, K1, g, "cuda")
    b = workloads.make_activation("student_t", M, K2, g, "cuda")
    want_q, want_sf = concat_reference(B, [a, b])
    xb = bits_of(torch.cat([a, b], dim=1))
    q_or, sf_or = oracle.mxfp4_quantize(xb)
    assert np.array_equal(want_q.cpu().numpy(), q_or)            # the reference itself against the oracle
    assert np.array_equal(want_sf.cpu().numpy(), oracle.mx_sf_swizzle(sf_or, K1 + K2))
    dest = (torch.full((M, (K1 + K2) // 2), 0xEE, dtype=torch.uint8, device="cuda"),
            torch.full((B.mxfp4_scale_bytes(M, K1 + K2),), 0xEE, dtype=torch.uint8, device="cuda"))
    B.mxfp4_quantize_into(b, dest, K1)
    assert torch.all(dest[0][:, :K1 // 2] == 0xEE)               # the other column range is untouched
    B.mxfp4_quantize_into(a, dest, 0)
    B.sol_last_device_status()
    assert torch.equal(dest[0], want_q)
    got_sf = dest[1].cpu().numpy()[mx_offsets(np.arange(M), K1 + K2)]
    assert np.array_equal(got_sf, sf_or)


@pytest.mark.parametrize("M,N,n_split,K,col0,dest_K", [(256, 512, 256, 64, 0, 256), (300, 896, 256, 256, 128, 1024),
                                                      (520, 768, 512, 512, 384, 640)])
def test_split_output_integer_exact_bit_for_bit(B, M, N, n_split, K, col0, dest_K):
    rng = np.random.default_rng(M + N + K)
    qx, sfx = pow2_mx(rng, M, K)
    qw, sfw = pow2_mx(rng, N, K)
    Y = oracle.mxfp4_linear(qx, sfx, qw, sfw)
    if np.abs(Y).max() * 4 >= 2 ** 24:
        pytest.skip("sum too large for an exact FP32 accumulator")
    part = N - n_split
    h_bits = oracle.round_bf16(Y[:, n_split:])
    q_ref, sf_ref = oracle.mxfp4_quantize(h_bits)
    dest = (torch.full((M, dest_K // 2), 0xEE, dtype=torch.uint8, device="cuda"),
            torch.full((B.mxfp4_scale_bytes(M, dest_K),), 0xEE, dtype=torch.uint8, device="cuda"))
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    y = B.mxfp4_linear_split_out(dev(qx), dev(oracle.mx_sf_swizzle(sfx, K)), dev(qw), dev(oracle.mx_sf_swizzle(sfw, K)),
                                 None, n_split, B.ACT_NONE, dest, col0, amax_out=amax)
    B.sol_last_device_status()
    assert np.array_equal(bits_of(y), oracle.round_bf16(Y[:, :n_split]))
    got_q = dest[0].cpu().numpy()
    assert np.array_equal(got_q[:, col0 // 2:(col0 + part) // 2], q_ref)
    untouched = np.ones(dest_K // 2, bool)
    untouched[col0 // 2:(col0 + part) // 2] = False
    assert np.all(got_q[:, untouched] == 0xEE)
    offs = mx_offsets(np.arange(M), dest_K)
    got_sf = dest[1].cpu().numpy()[offs]
    assert np.array_equal(got_sf[:, col0 // 32:(col0 + part) // 32], sf_ref)
    keep = np.ones(dest_K // 32, bool)
    keep[col0 // 32:(col0 + part) // 32] = False
    assert np.all(got_sf[:, keep] == 0xEE)
    assert amax.item() == np.abs(oracle.bits_to_f64(h_bits)).max()


def test_single_stream_chain_in_mxfp4(B):
    # split linear (q/k/v BF16 | GELU(MLP) as MXFP4 into the concat) + slice quantizer for the attention part,
    # then the second linear on the concatenated MXFP4 tensor: equal to the unfused chain built from the
    # entries checked above (mxfp4_linear, torch's tanh-GELU rounded to BF16 is NOT used: the quantized part is
    # compared through its dequantized values against the oracle's FP64 GELU within the format's step)
    M, K, n_split, n_mlp, attn_w, N2 = 384, 512, 768, 1024, 256, 256
    N = n_split + n_mlp
    g = torch.Generator(device="cuda").manual_seed(5)
    X = workloads.make_activation("student_t", M, K, g, "cuda")
    W1 = (torch.randn(N, K, generator=g, device="cuda") * K ** -0.5).to(torch.bfloat16)
    b1 = (torch.randn(N, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    attn = workloads.make_activation("student_t", M, attn_w, g, "cuda")
    xq, w1q = B.mxfp4_quantize(X), B.mxfp4_quantize(W1)
    dest_K = attn_w + n_mlp
    dest = (torch.zeros((M, dest_K // 2), dtype=torch.uint8, device="cuda"),
            torch.zeros(B.mxfp4_scale_bytes(M, dest_K), dtype=torch.uint8, device="cuda"))
    y_qkv = B.mxfp4_linear_split_out(*xq, *w1q, b1, n_split, B.ACT_GELU_TANH, dest, attn_w)
    B.mxfp4_quantize_into(attn, dest, 0)
    B.sol_last_device_status()
    y_full = B.mxfp4_linear(*xq, *w1q, b1)
    assert torch.equal(y_qkv, y_full[:, :n_split].contiguous())
    # the attention slice is bit for bit the quantizer's output on that slice
    aq, asf = B.mxfp4_quantize(attn)
    assert torch.equal(dest[0][:, :attn_w // 2], aq)
    # the MLP slice against the oracle's FP64 GELU of the FP64 linear
    qx, sfx = oracle.mxfp4_quantize(bits_of(X))
    qw, sfw = oracle.mxfp4_quantize(bits_of(W1))
    Y = oracle.mxfp4_linear(qx, sfx, qw, sfw, bits_of(b1))[:, n_split:]
    H = oracle.gelu_tanh(Y)
    sf_rm = dest[1].cpu().numpy()[mx_offsets(np.arange(M), dest_K)][:, attn_w // 32:]
    deq = oracle.mxfp4_dequantize(dest[0][:, attn_w // 2:].contiguous().cpu().numpy(), sf_rm)
    scale = np.repeat(np.ldexp(1.0, sf_rm.astype(np.int32) - 127), 32, axis=1)
    tol = 1.2 * oracle.linear_tolerance(Y) + 2.0 ** -8 * np.abs(H)
    reach = np.maximum(1.0 * scale, np.abs(H) - 6.0 * scale)
    assert np.all(np.abs(deq - H) <= reach * (1 + 2.0 ** -6) + tol)
