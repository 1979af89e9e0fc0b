"""GPU parity: BF16 and NVFP4 linears vs the FP64 oracle, through the C ABI.

Tolerance (every output): |gpu - oracle| <= 2^-7 |oracle| + 1e-4 rms(oracle row).
Integer-exact cases (power-of-two scales, small K) must match bf16_rne(oracle) bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_06916_b200 import workloads
from tests.helpers import bits_of, check_linear, sample_rows, unswizzle_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06916_b200 import binding
    binding.lib()
    return binding


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def upload_quantized(q: np.ndarray, sf: np.ndarray, K: int, T: float):
    return dev(q), dev(oracle.sf_swizzle(sf, K)), torch.tensor([T], dtype=torch.float32, device="cuda")


def random_pow2_quantized(rng, rows, K, exps=(-2, 2)):
    q = rng.integers(0, 256, size=(rows, K // 2), dtype=np.uint8)
    e = rng.integers(exps[0], exps[1] + 1, size=(rows, K // 16))
    return q, ((e + 7) << 3).astype(np.uint8)


# ------------------------------------------------------------------ BF16 linear
@pytest.mark.parametrize("M,N,K", [(256, 512, 512), (128, 256, 64), (200, 136, 96), (130, 264, 2240), (1, 8, 32)])
def test_bf16_linear_small_shapes_full_compare(B, M, N, K):
    g = torch.Generator(device="cuda").manual_seed(M * 7 + N)
    x = torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16)
    w = (torch.randn(N, K, generator=g, device="cuda") * K ** -0.5).to(torch.bfloat16)
    b = (torch.randn(N, generator=g, device="cuda") * 0.1).to(torch.bfloat16)
    for bias in (b, None):
        y = B.bf16_linear(x, w, bias)
        B.sol_last_device_status()
        Y = oracle.bf16_linear(bits_of(x), bits_of(w), None if bias is None else bits_of(bias))
        check_linear(bits_of(y), Y, f"bf16 {M}x{N}x{K} bias={bias is not None}")


def test_bf16_linear_integer_exact(B):
    g = torch.Generator(device="cuda").manual_seed(5)
    M, N, K = 384, 520, 320
    x = torch.randint(-4, 5, (M, K), generator=g, device="cuda").to(torch.bfloat16)
    w = torch.randint(-4, 5, (N, K), generator=g, device="cuda").to(torch.bfloat16)
    y = B.bf16_linear(x, w)
    Y = oracle.bf16_linear(bits_of(x), bits_of(w))
    assert np.array_equal(bits_of(y), oracle.round_bf16(Y))


def test_bf16_linear_row_pitches(B):
    g = torch.Generator(device="cuda").manual_seed(6)
    M, N, K = 192, 264, 160
    xf = torch.randn(M, K + 16, generator=g, device="cuda").to(torch.bfloat16)
    wf = torch.randn(N, K + 8, generator=g, device="cuda").to(torch.bfloat16)
    yf = torch.full((M, N + 24), 7.0, dtype=torch.bfloat16, device="cuda")
    B.bf16_linear(xf[:, :K], wf[:, :K], None, out=yf[:, :N])
    Y = oracle.bf16_linear(bits_of(xf[:, :K]), bits_of(wf[:, :K]))
    check_linear(bits_of(yf[:, :N]), Y, "pitched")
    assert torch.all(yf[:, N:] == 7.0)  # nothing written past N


# ------------------------------------------------------------------ NVFP4 linear
@pytest.mark.parametrize("M,N,K", [(128, 192, 64), (128, 192, 256), (256, 384, 512), (130, 200, 96), (64, 8, 32),
                                   (300, 456, 448)])
def test_nvfp4_linear_integer_exact(B, M, N, K):
    rng = np.random.default_rng(M + N + K)
    qx, sfx = random_pow2_quantized(rng, M, K)
    qw, sfw = random_pow2_quantized(rng, N, K)
    Y = oracle.nvfp4_linear(qx, sfx, 1.0, qw, sfw, 1.0)
    y = B.nvfp4_linear(*upload_quantized(qx, sfx, K, 1.0), *upload_quantized(qw, sfw, K, 1.0))
    B.sol_last_device_status()
    got, want = bits_of(y), oracle.round_bf16(Y)
    bad = got != want
    assert not bad.any(), (f"{int(bad.sum())} of {bad.size} differ; rows {np.unique(np.argwhere(bad)[:, 0])[:10]} "
                           f"cols {np.unique(np.argwhere(bad)[:, 1])[:10]}")


def test_nvfp4_scale_and_nibble_placement(B):
    """One non-zero row of X whose 16-element blocks carry distinct power-of-two scales, against
    one-hot rows of W: every output isolates one (row, block) scale and one nibble position."""
    M, N, K = 128, 192, 512
    for row in (0, 37, 127):
        qx = np.zeros((M, K // 2), np.uint8)
        sfx = np.full((M, K // 16), 0x38, np.uint8)
        qx[row, :] = 0x22                                  # every element +1.0
        sfx[row, :] = ((np.arange(K // 16) % 8) + 4) << 3  # 2^(b%8 - 3)
        qw = np.zeros((N, K // 2), np.uint8)
        sfw = np.full((N, K // 16), 0x38, np.uint8)
        ks = (np.arange(N) * 37 + 5) % K                   # W row n selects element ks[n]
        for n, k in enumerate(ks):
            qw[n, k // 2] = 0x2 << (4 * (k & 1))
            sfw[n, k // 16] = ((n % 5) + 5) << 3           # 2^(n%5 - 2)
        Y = oracle.nvfp4_linear(qx, sfx, 1.0, qw, sfw, 1.0)
        y = B.nvfp4_linear(*upload_quantized(qx, sfx, K, 1.0), *upload_quantized(qw, sfw, K, 1.0))
        assert np.array_equal(bits_of(y), oracle.round_bf16(Y)), f"row {row}"
        assert np.count_nonzero(Y) == N


def test_nvfp4_linear_config1_full(B):
    X, W, bias = workloads.make_layer(workloads.CONFIG_SINGLE, 0, "cuda")
    xb, wb = bits_of(X), bits_of(W)
    Tx, Tw = oracle.tensor_scale(xb), oracle.tensor_scale(wb)
    qx, sfx = oracle.quantize(xb, Tx)
    qw, sfw = oracle.quantize(wb, Tw)
    Y = oracle.nvfp4_linear(qx, sfx, Tx, qw, sfw, Tw, bits_of(bias))
    K = X.shape[1]
    y = B.nvfp4_linear(*upload_quantized(qx, sfx, K, Tx), *upload_quantized(qw, sfw, K, Tw), bias)
    check_linear(bits_of(y), Y, "config1 nvfp4_linear")
    # fused entry: quantize on the GPU, then the same GEMM
    wq, wsf, wts = B.nvfp4_quantize_weight(W)
    y2 = B.nvfp4_quantize_linear(X, wq, wsf, wts, bias)
    B.sol_last_device_status()
    assert torch.equal(y, y2)


def run_layer_sampled(B, cfg, index, M=None):
    layer = cfg.layers[index]
    X, W, bias = workloads.make_layer(cfg, index, "cuda", M=M)
    Mrows, K, N = X.shape[0], layer.K, layer.N
    rows = sample_rows(Mrows, seed=index)
    # NVFP4: quantize on the GPU (bit-exactness is covered elsewhere), oracle on the sampled rows
    wq, wsf, wts = B.nvfp4_quantize_weight(W)
    xts = B.sol_amax_bf16(X)
    xq, xsf = B.nvfp4_quantize(X, xts)
    y = B.nvfp4_linear(xq, xsf, xts, wq, wsf, wts, bias)
    y_fused = B.nvfp4_quantize_linear(X, wq, wsf, wts, bias)
    y_bf16 = B.bf16_linear(X, W, bias)
    B.sol_last_device_status()
    assert torch.equal(y, y_fused)
    rows_t = torch.from_numpy(rows).cuda()
    qx_s = xq[rows_t].cpu().numpy()
    sfx_s = unswizzle_rows(xsf.cpu().numpy(), rows, K)
    sfw_rm = unswizzle_rows(wsf.cpu().numpy(), np.arange(N), K)
    Y = oracle.nvfp4_linear(qx_s, sfx_s, xts.item(), wq.cpu().numpy(), sfw_rm, wts.item(), bits_of(bias))
    check_linear(bits_of(y[rows_t]), Y, f"{cfg.name}/{layer.name} nvfp4")
    Yb = oracle.bf16_linear(bits_of(X[rows_t]), bits_of(W), bits_of(bias))
    check_linear(bits_of(y_bf16[rows_t]), Yb, f"{cfg.name}/{layer.name} bf16")


@pytest.mark.parametrize("index", range(4))
def test_sana_shaped_layers_sampled_rows(B, index):
    run_layer_sampled(B, workloads.CONFIG_SANA, index)


@pytest.mark.parametrize("index", range(4))
def test_sd35_shaped_layers_sampled_rows(B, index):
    run_layer_sampled(B, workloads.CONFIG_SD35, index)


@pytest.mark.parametrize("index", range(6))
def test_flux_shaped_layers_sampled_rows(B, index):
    run_layer_sampled(B, workloads.CONFIG_FLUX, index)


def test_host_buffer_entry_matches_device_entry(B):
    cfg = workloads.CONFIG_SANA
    X, W, bias = workloads.make_layer(cfg, 1, "cuda", M=2500)
    wq, wsf, wts = B.nvfp4_quantize_weight(W)
    want = B.nvfp4_quantize_linear(X, wq, wsf, wts, bias)
    xh = torch.empty(X.shape[0], X.shape[1] + 8, dtype=torch.bfloat16).pin_memory()[:, :X.shape[1]]
    xh.copy_(X)
    yh = torch.zeros(want.shape[0], want.shape[1] + 16, dtype=torch.bfloat16).pin_memory()[:, :want.shape[1]]
    ws = torch.empty(B.linear_workspace_bytes(*want.shape, X.shape[1]), dtype=torch.uint8, device="cuda")
    B.nvfp4_quantize_linear_host(xh, wq, wsf, wts, bias, yh, torch.empty_like(X), torch.empty_like(want), ws)
    B.sol_last_device_status()
    assert torch.equal(yh, want.cpu())


def test_deterministic_run_to_run(B):
    cfg = workloads.CONFIG_SANA
    X, W, bias = workloads.make_layer(cfg, 1, "cuda", M=4096)
    wq, wsf, wts = B.nvfp4_quantize_weight(W)
    a = B.nvfp4_quantize_linear(X, wq, wsf, wts, bias)
    b = B.nvfp4_quantize_linear(X, wq, wsf, wts, bias)
    assert torch.equal(a, b)
    assert torch.equal(B.bf16_linear(X, W, bias), B.bf16_linear(X, W, bias))


@pytest.mark.parametrize("index", [1, 5])  # d_proj (K = 3072) and s_out (K = 15360), full M = 36864
def test_flux_layers_every_output_against_library_matmul_screen(B, index):
    # secondary screen with full coverage: a library BF16 matmul (FP32 accumulation) on the
    # dequantized operands; the oracle itself covers sampled rows of the same launches above
    from tests.helpers import dequantize_on_device
    cfg = workloads.CONFIG_FLUX
    layer = cfg.layers[index]
    X, W, bias = workloads.make_layer(cfg, index, "cuda")
    wq, wsf, wts = B.nvfp4_quantize_weight(W)
    xts = B.sol_amax_bf16(X)
    xq, xsf = B.nvfp4_quantize(X, xts)
    y = B.nvfp4_linear(xq, xsf, xts, wq, wsf, wts, bias)
    B.sol_last_device_status()
    xd = dequantize_on_device(xq, xsf, layer.M, layer.K)
    wd = dequantize_on_device(wq, wsf, layer.N, layer.K)
    del X, W, xq, xsf
    alpha = (xts * wts).item()
    worst = 0.0
    for r0 in range(0, layer.M, 4096):
        acc = torch.matmul(xd[r0:r0 + 4096], wd.t()).float()      # BF16 result of an FP32 accumulation
        ref = acc * alpha + bias.float()[None, :]
        got = y[r0:r0 + 4096].float()
        # the screen's own BF16 rounding of acc adds 2^-9 relative; the product bound stays 2^-7
        tol = 2.0 ** -7 * ref.abs() + 1e-4 * ref.pow(2).mean(dim=1, keepdim=True).sqrt() + 2.0 ** -8 * (acc * alpha).abs()
        err = (got - ref).abs()
        assert bool((err <= tol).all()), f"rows {r0}..: {(err > tol).sum().item()} outputs off"
        worst = max(worst, float((err / tol.clamp_min(1e-30)).max()))
    assert worst <= 1.0


def test_delayed_scale_entry(B):
    # with the same T the delayed entry equals quantize + linear bit for bit, its by-product is the
    # exact amax of X, and rolling the state gives the tensor scale the dynamic path would compute
    X, W, bias = workloads.make_layer(workloads.CONFIG_SANA, 1, "cuda", M=1000)
    wq, wsf, wts = B.nvfp4_quantize_weight(W)
    state = torch.tensor([0.05, 0.0], dtype=torch.float32, device="cuda")
    y = B.nvfp4_quantize_linear_delayed(X, wq, wsf, wts, bias, state)
    ts = state[:1].clone()
    xq, xsf = B.nvfp4_quantize(X, ts)
    assert torch.equal(y, B.nvfp4_linear(xq, xsf, ts, wq, wsf, wts, bias))
    assert state[0].item() == np.float32(0.05)
    amax = np.abs(oracle.bits_to_f64(bits_of(X))).max()
    assert state[1].item() == amax
    B.sol_roll_tensor_scale(state)
    assert state[0].item() == oracle.tensor_scale(bits_of(X)) and state[1].item() == 0.0
    # second step with the rolled scale = the dynamic entry on the same X
    y2 = B.nvfp4_quantize_linear_delayed(X, wq, wsf, wts, bias, state)
    assert torch.equal(y2, B.nvfp4_quantize_linear(X, wq, wsf, wts, bias))
    B.sol_last_device_status()
