"""GPU parity: the NVFP4 linear whose output is already quantized for the next linear.

The accumulation order inside the tensor core is not the oracle's, so h = bf16(act(y)) can differ
from the oracle's in its last place on a small share of the elements and a quantized code can
then differ too.  What is unique is checked bit for bit (integer-exact inputs, where both sides
hold the same h); elsewhere the output must be VALID: the scale byte is the oracle's or its
neighbour, almost all codes are the oracle's, and every dequantized value lies within the
quantizer's rounding interval (at the emitted scale) around the oracle's FP64 activation, widened
by the linear's tolerance.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_06916_b200 import workloads
from tests.helpers import bits_of, sample_rows, unswizzle_rows

pytestmark = pytest.mark.gpu

GRID = np.array([0, .5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)
HALF_WIDTH = 0.5 * np.array([.5, .5, .5, .5, 1, 1, 2, 2], dtype=np.float64)   # widest half gap next to each magnitude


@pytest.fixture(scope="module")
def B():
    from paper_2604_06916_b200 import binding
    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def upload(q, sf, K, T):
    return dev(q), dev(oracle.sf_swizzle(sf, K)), torch.tensor([T], dtype=torch.float32, device="cuda")


def nibbles(q: np.ndarray) -> np.ndarray:
    out = np.empty((q.shape[0], q.shape[1] * 2), np.uint8)
    out[:, 0::2] = q & 0xF
    out[:, 1::2] = q >> 4
    return out


def scale_values(sf: np.ndarray) -> np.ndarray:
    table = np.array([oracle.e4m3_decode(c) for c in range(128)])
    return table[sf]


def check_valid(hq, hsf_rm, Y, H, q_star, sf_star, T, min_code_match, act):
    codes, codes_star = nibbles(hq), nibbles(q_star)
    assert (hsf_rm == sf_star).mean() >= 0.995
    assert np.abs(hsf_rm.astype(np.int32) - sf_star.astype(np.int32)).max() <= 1
    assert (codes == codes_star).mean() >= min_code_match, (codes == codes_star).mean()
    s = np.repeat(scale_values(hsf_rm), 16, axis=1) * float(T)
    mag = codes & 7
    val = np.where(codes & 8, -GRID[mag], GRID[mag]) * s
    rms = np.sqrt(np.mean(Y * Y, axis=1, keepdims=True))
    slope = 1.2 if act else 1.0                      # |gelu'| < 1.13
    tol = slope * (2.0 ** -7 * np.abs(Y) + 1e-4 * rms) + 2.0 ** -8 * np.abs(H)
    bound = HALF_WIDTH[mag] * s * (1 + 2.0 ** -6) + tol
    err = np.abs(val - H)
    bad = err > bound
    assert not bad.any(), f"{int(bad.sum())} of {bad.size} dequantized outputs outside their rounding interval"


@pytest.mark.parametrize("M,N,K", [(256, 256, 64), (128, 192, 256), (300, 448, 448), (64, 64, 32), (520, 1024, 512)])
def test_integer_exact_inputs_bit_for_bit(B, M, N, K):
    rng = np.random.default_rng(M * 3 + N + K)
    qx = rng.integers(0, 256, size=(M, K // 2), dtype=np.uint8)
    qw = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    sfx = ((rng.integers(-2, 3, size=(M, K // 16)) + 7) << 3).astype(np.uint8)
    sfw = ((rng.integers(-2, 3, size=(N, K // 16)) + 7) << 3).astype(np.uint8)
    Y = oracle.nvfp4_linear(qx, sfx, 1.0, qw, sfw, 1.0)
    T_out = float(oracle.tensor_scale(oracle.round_bf16(Y)))
    H, h, q_star, sf_star = oracle.nvfp4_linear_quantized(qx, sfx, 1.0, qw, sfw, 1.0, None, oracle.ACT_NONE, T_out)
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    ts_out = torch.tensor([T_out], dtype=torch.float32, device="cuda")
    hq, hsf = B.nvfp4_linear_quantized_out(*upload(qx, sfx, K, 1.0), *upload(qw, sfw, K, 1.0), None, B.ACT_NONE,
                                           ts_out, amax_out=amax)
    B.sol_last_device_status()
    assert np.array_equal(hq.cpu().numpy(), q_star)
    assert np.array_equal(hsf.cpu().numpy().ravel(), oracle.sf_swizzle(sf_star, N).ravel())   # padding rows are 0
    assert amax.item() == np.abs(oracle.bits_to_f64(h)).max()
    # the running maximum only grows
    amax.fill_(1e30)
    B.nvfp4_linear_quantized_out(*upload(qx, sfx, K, 1.0), *upload(qw, sfw, K, 1.0), None, B.ACT_NONE, ts_out,
                                 amax_out=amax)
    assert amax.item() == np.float32(1e30)


@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("M,N,K", [(384, 512, 1024), (1000, 320, 96)])
def test_general_inputs_valid_output(B, act, M, N, K):
    g = torch.Generator(device="cuda").manual_seed(M + N + K + act)
    X = workloads.make_activation("student_t", M, K, g, "cuda")
    W = (torch.randn(N, K, generator=g, device="cuda") * K ** -0.5).to(torch.bfloat16)
    bias = (torch.randn(N, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    xb, wb, bb = bits_of(X), bits_of(W), bits_of(bias)
    Tx, Tw = oracle.tensor_scale(xb), oracle.tensor_scale(wb)
    qx, sfx = oracle.quantize(xb, Tx)
    qw, sfw = oracle.quantize(wb, Tw)
    Y = oracle.nvfp4_linear(qx, sfx, Tx, qw, sfw, Tw, bb)
    Hfull = oracle.gelu_tanh(Y) if act else Y
    T_out = float(oracle.tensor_scale(oracle.round_bf16(Hfull)))
    H, h, q_star, sf_star = oracle.nvfp4_linear_quantized(qx, sfx, Tx, qw, sfw, Tw, bb, act, T_out)
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    hq, hsf = B.nvfp4_linear_quantized_out(*upload(qx, sfx, K, Tx), *upload(qw, sfw, K, Tw), bias, act,
                                           torch.tensor([T_out], dtype=torch.float32, device="cuda"), amax_out=amax)
    B.sol_last_device_status()
    hsf_rm = unswizzle_rows(hsf.cpu().numpy().ravel(), np.arange(M), N)
    check_valid(hq.cpu().numpy(), hsf_rm, Y, H, q_star, sf_star, T_out, 0.99, act)
    want_amax = np.abs(oracle.bits_to_f64(h)).max()
    assert abs(amax.item() - want_amax) <= 2.0 ** -7 * want_amax
    # feeding the fused output to the next linear gives what the oracle's chain gives, up to the
    # effect of the few codes and scale bytes of h that may legitimately differ (each moves one
    # term of a row's sum by a grid step: a few per cent of the row's rms in total)
    W2 = (torch.randn(256, N, generator=g, device="cuda") * N ** -0.5).to(torch.bfloat16)
    w2q, w2sf, w2ts = B.nvfp4_quantize_weight(W2)
    y2 = B.nvfp4_linear(hq, hsf, torch.tensor([T_out], dtype=torch.float32, device="cuda"), w2q, w2sf, w2ts)
    qw2, sfw2 = oracle.quantize(bits_of(W2), oracle.tensor_scale(bits_of(W2)))
    Y2 = oracle.nvfp4_linear(q_star, sf_star, T_out, qw2, sfw2, oracle.tensor_scale(bits_of(W2)))
    err = np.abs(oracle.bits_to_f64(bits_of(y2)) - Y2)
    rms = np.sqrt(np.mean(Y2 * Y2, axis=1, keepdims=True))
    assert np.all(err <= 2.0 ** -4 * np.abs(Y2) + 0.1 * rms)
    assert np.mean(err / rms) < 0.01


def test_flux_mlp_in_full_size_sampled_rows(B):
    # FLUX double-stream MLP-in (36864 x 3072 -> 12288) with GELU, the launch the benchmark times
    cfg = workloads.CONFIG_FLUX
    X, W, bias = workloads.make_layer(cfg, 2, "cuda")
    M, K, N = X.shape[0], X.shape[1], W.shape[0]
    wq, wsf, wts = B.nvfp4_quantize_weight(W)
    xts = B.sol_amax_bf16(X)
    xq, xsf = B.nvfp4_quantize(X, xts)
    rows = sample_rows(M, seed=7)
    rows_t = torch.from_numpy(rows).cuda()
    sfw_rm = unswizzle_rows(wsf.cpu().numpy(), np.arange(N), K)
    qx_s, sfx_s = xq[rows_t].cpu().numpy(), unswizzle_rows(xsf.cpu().numpy(), rows, K)
    Y = oracle.nvfp4_linear(qx_s, sfx_s, xts.item(), wq.cpu().numpy(), sfw_rm, wts.item(), bits_of(bias))
    Hs = oracle.gelu_tanh(Y)
    T_out = float(np.float32(np.abs(Hs).max() * 1.05 / 2688.0))    # a calibrated scale with 5 % headroom
    H, h, q_star, sf_star = oracle.nvfp4_linear_quantized(qx_s, sfx_s, xts.item(), wq.cpu().numpy(), sfw_rm,
                                                          wts.item(), bits_of(bias), 1, T_out)
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    hq, hsf = B.nvfp4_linear_quantized_out(xq, xsf, xts, wq, wsf, wts, bias, B.ACT_GELU_TANH,
                                           torch.tensor([T_out], dtype=torch.float32, device="cuda"), amax_out=amax)
    B.sol_last_device_status()
    hsf_rm = unswizzle_rows(hsf.cpu().numpy().ravel(), rows, N)
    check_valid(hq[rows_t].cpu().numpy(), hsf_rm, Y, H, q_star, sf_star, T_out, 0.99, 1)
    assert amax.item() >= np.abs(oracle.bits_to_f64(h)).max() * (1 - 2.0 ** -7)


def test_rejects_bad_arguments(B):
    z = torch.zeros(64 * 32, dtype=torch.uint8, device="cuda")
    t = torch.ones(1, dtype=torch.float32, device="cuda")
    with pytest.raises(B.SolError):   # N must be a multiple of 64
        B.lib().nvfp4_linear_quantized_out  # symbol exists
        B._check(B.lib().nvfp4_linear_quantized_out(z.data_ptr(), z.data_ptr(), t.data_ptr(), z.data_ptr(), z.data_ptr(),
                                                    t.data_ptr(), None, 0, t.data_ptr(), z.data_ptr(), z.data_ptr(), None,
                                                    64, 96, 64, None), "nvfp4_linear_quantized_out")


def test_quantize_into_slice_bit_exact(B):
    # two BF16 parts quantized into one wider tensor equal the oracle's quantizer on their concatenation
    g = torch.Generator(device="cuda").manual_seed(21)
    M, K1, K2 = 300, 192, 448
    X1 = workloads.make_activation("student_t", M, K1, g, "cuda")
    X2 = workloads.make_activation("outlier", M, K2, g, "cuda")
    cat_bits = np.concatenate([bits_of(X1), bits_of(X2)], axis=1)
    T = oracle.tensor_scale(cat_bits)
    want_q, want_sf = oracle.quantize(cat_bits, T)
    K = K1 + K2
    hq = torch.full((M, K // 2), 0xEE, dtype=torch.uint8, device="cuda")
    hsf = torch.zeros(B.scale_bytes(M, K), dtype=torch.uint8, device="cuda")
    ts = torch.tensor([T], dtype=torch.float32, device="cuda")
    B.nvfp4_quantize_into(X2, ts, (hq, hsf), K1)
    assert torch.all(hq[:, : K1 // 2] == 0xEE)                 # the other column range is untouched
    B.nvfp4_quantize_into(X1, ts, (hq, hsf), 0)
    assert np.array_equal(hq.cpu().numpy(), want_q)
    assert np.array_equal(hsf.cpu().numpy(), oracle.sf_swizzle(want_sf, K))


@pytest.mark.parametrize("M,N,n_split,K,col0,dest_K", [(256, 512, 256, 64, 0, 256), (300, 832, 256, 256, 128, 768),
                                                       (520, 1024, 512, 512, 64, 640)])
def test_split_output_integer_exact_bit_for_bit(B, M, N, n_split, K, col0, dest_K):
    rng = np.random.default_rng(M + N + K)
    qx = rng.integers(0, 256, size=(M, K // 2), dtype=np.uint8)
    qw = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    sfx = ((rng.integers(-2, 3, size=(M, K // 16)) + 7) << 3).astype(np.uint8)
    sfw = ((rng.integers(-2, 3, size=(N, K // 16)) + 7) << 3).astype(np.uint8)
    Y = oracle.nvfp4_linear(qx, sfx, 1.0, qw, sfw, 1.0)
    h = oracle.round_bf16(Y[:, n_split:])
    T_out = float(oracle.tensor_scale(h))
    q_star, sf_star = oracle.quantize(h, T_out)
    part = N - n_split
    hq = torch.full((M, dest_K // 2), 0xEE, dtype=torch.uint8, device="cuda")
    hsf = torch.full((B.scale_bytes(M, dest_K),), 0xDD, dtype=torch.uint8, device="cuda")
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    y = B.nvfp4_linear_split_out(*upload(qx, sfx, K, 1.0), *upload(qw, sfw, K, 1.0), None, n_split, B.ACT_NONE,
                                 torch.tensor([T_out], dtype=torch.float32, device="cuda"), (hq, hsf), col0,
                                 amax_out=amax)
    B.sol_last_device_status()
    assert np.array_equal(bits_of(y), oracle.round_bf16(Y[:, :n_split]))
    got_q = hq.cpu().numpy()
    assert np.array_equal(got_q[:, col0 // 2:(col0 + part) // 2], q_star)
    untouched = np.ones(dest_K // 2, bool)
    untouched[col0 // 2:(col0 + part) // 2] = False
    assert np.all(got_q[:, untouched] == 0xEE)
    sf_all = unswizzle_rows(hsf.cpu().numpy(), np.arange(M), dest_K)
    assert np.array_equal(sf_all[:, col0 // 16:(col0 + part) // 16], sf_star)
    mask = np.ones(dest_K // 16, bool)
    mask[col0 // 16:(col0 + part) // 16] = False
    assert np.all(sf_all[:, mask] == 0xDD)
    assert amax.item() == np.abs(oracle.bits_to_f64(h)).max()


def test_single_stream_block_chain_against_oracle(B):
    # first linear: q/k/v part in BF16 + GELU(MLP part) quantized into the concat buffer at column 256;
    # a BF16 "attention output" quantized into columns [0, 256); second linear on the concat buffer
    g = torch.Generator(device="cuda").manual_seed(33)
    M, K, n_split, n_mlp, attn_w, N2 = 384, 512, 768, 1024, 256, 256
    N = n_split + n_mlp
    X = workloads.make_activation("student_t", M, K, g, "cuda")
    W1 = (torch.randn(N, K, generator=g, device="cuda") * K ** -0.5).to(torch.bfloat16)
    b1 = (torch.randn(N, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    attn = (torch.randn(M, attn_w, generator=g, device="cuda") * 0.5).to(torch.bfloat16)
    W2 = (torch.randn(N2, attn_w + n_mlp, generator=g, device="cuda") * (attn_w + n_mlp) ** -0.5).to(torch.bfloat16)
    xb, w1b = bits_of(X), bits_of(W1)
    Tx, Tw1 = oracle.tensor_scale(xb), oracle.tensor_scale(w1b)
    qx, sfx = oracle.quantize(xb, Tx)
    qw1, sfw1 = oracle.quantize(w1b, Tw1)
    Y1 = oracle.nvfp4_linear(qx, sfx, Tx, qw1, sfw1, Tw1, bits_of(b1))
    H = oracle.gelu_tanh(Y1[:, n_split:])
    cat = np.concatenate([bits_of(attn), oracle.round_bf16(H)], axis=1)
    T_cat = float(oracle.tensor_scale(cat))
    q_cat, sf_cat = oracle.quantize(cat, T_cat)
    dest_K = attn_w + n_mlp
    hq = torch.zeros((M, dest_K // 2), dtype=torch.uint8, device="cuda")
    hsf = torch.zeros(B.scale_bytes(M, dest_K), dtype=torch.uint8, device="cuda")
    ts = torch.tensor([T_cat], dtype=torch.float32, device="cuda")
    y_qkv = B.nvfp4_linear_split_out(*upload(qx, sfx, K, Tx), *upload(qw1, sfw1, K, Tw1), b1, n_split, B.ACT_GELU_TANH, ts,
                                     (hq, hsf), attn_w)
    B.nvfp4_quantize_into(attn, ts, (hq, hsf), 0)
    B.sol_last_device_status()
    from tests.helpers import check_linear
    check_linear(bits_of(y_qkv), Y1[:, :n_split], "qkv part")
    got_q = hq.cpu().numpy()
    sf_rm = unswizzle_rows(hsf.cpu().numpy(), np.arange(M), dest_K)
    assert np.array_equal(got_q[:, : attn_w // 2], q_cat[:, : attn_w // 2])               # BF16 part: bit-exact
    assert np.array_equal(sf_rm[:, : attn_w // 16], sf_cat[:, : attn_w // 16])
    check_valid(got_q[:, attn_w // 2:], sf_rm[:, attn_w // 16:], Y1[:, n_split:], H, q_cat[:, attn_w // 2:],
                sf_cat[:, attn_w // 16:], T_cat, 0.99, 1)
    # second linear on the concat buffer against the oracle's chain
    w2q, w2sf, w2ts = B.nvfp4_quantize_weight(W2)
    y2 = B.nvfp4_linear(hq, hsf, ts, w2q, w2sf, w2ts)
    Tw2 = oracle.tensor_scale(bits_of(W2))
    qw2, sfw2 = oracle.quantize(bits_of(W2), Tw2)
    Y2 = oracle.nvfp4_linear(q_cat, sf_cat, T_cat, qw2, sfw2, Tw2)
    err = np.abs(oracle.bits_to_f64(bits_of(y2)) - Y2)
    rms = np.sqrt(np.mean(Y2 * Y2, axis=1, keepdims=True))
    assert np.all(err <= 2.0 ** -4 * np.abs(Y2) + 0.1 * rms) and np.mean(err / rms) < 0.01
