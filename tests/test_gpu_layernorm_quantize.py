"""GPU parity: layer norm + modulation fused with the NVFP4 quantizer, against the FP64 oracle.

The kernel's FP32 statistics differ from the oracle's FP64 ones in the last bits, so h = bf16(y) can
differ in its last place on a small share of the elements; as for the quantizing GEMM epilogue the
output is checked for validity: scale bytes equal on >= 99.5 % of the blocks and never more than
one code apart, codes equal on >= 99 %, every dequantized value inside the quantizer's rounding
interval (at the emitted scale) around the oracle's y, widened by 2^-8 |y| for the BF16 rounding
and 1e-5 (|y| + 1) for the FP32 statistics.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_06916_b200 import workloads
from tests.helpers import bits_of, unswizzle_rows

pytestmark = pytest.mark.gpu

GRID = np.array([0, .5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)
HALF_WIDTH = 0.5 * np.array([.5, .5, .5, .5, 1, 1, 2, 2], dtype=np.float64)


@pytest.fixture(scope="module")
def B():
    from paper_2604_06916_b200 import binding
    binding.lib()
    return binding


def nibbles(q):
    out = np.empty((q.shape[0], q.shape[1] * 2), np.uint8)
    out[:, 0::2] = q & 0xF
    out[:, 1::2] = q >> 4
    return out


def run_case(B, M, K, rps, seed, pad=0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    big = workloads.make_activation("student_t", M, K + pad, g, "cuda") * 1.7 + 0.3
    x = big[:, :K]
    S = (M + rps - 1) // rps
    scale = (torch.randn(S, K, generator=g, device="cuda") * 0.3).to(torch.bfloat16)
    shift = (torch.randn(S, K, generator=g, device="cuda") * 0.2).to(torch.bfloat16)
    xb = bits_of(x.contiguous())
    Yfull = oracle.layernorm_modulate(xb, bits_of(scale), bits_of(shift), rps)
    T = float(oracle.tensor_scale(oracle.round_bf16(Yfull)))
    Y, h, q_star, sf_star = oracle.layernorm_modulate_quantized(xb, bits_of(scale), bits_of(shift), rps, T)
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    ts = torch.tensor([T], dtype=torch.float32, device="cuda")
    q, sf = B.nvfp4_layernorm_quantize(x, scale, shift, rps, ts, amax_out=amax)
    torch.cuda.synchronize()
    sf_np = sf.cpu().numpy()
    sf_rm = unswizzle_rows(sf_np, np.arange(M), K)
    codes, codes_star = nibbles(q.cpu().numpy()), nibbles(q_star)
    assert (sf_rm == sf_star).mean() >= 0.995
    assert np.abs(sf_rm.astype(np.int32) - sf_star.astype(np.int32)).max() <= 1
    assert (codes == codes_star).mean() >= 0.99
    table = np.array([oracle.e4m3_decode(c) for c in range(128)])
    s = np.repeat(table[sf_rm], 16, axis=1) * T
    mag = codes & 7
    val = np.where(codes & 8, -GRID[mag], GRID[mag]) * s
    bound = HALF_WIDTH[mag] * s * (1 + 2.0 ** -6) + 2.0 ** -8 * np.abs(Y) + 1e-5 * (np.abs(Y) + 1)
    assert np.all(np.abs(val - Y) <= bound)
    want_amax = np.abs(oracle.bits_to_f64(h)).max()
    assert abs(amax.item() - want_amax) <= 2.0 ** -7 * want_amax
    # padding rows of the last 128-row scale chunk are zero
    mask = np.ones(sf_np.size, bool)
    from tests.helpers import swizzled_offsets
    mask[swizzled_offsets(np.arange(M), K).ravel()] = False
    assert np.all(sf_np[mask] == 0)
    return (sf_rm == sf_star).mean(), (codes == codes_star).mean()


@pytest.mark.parametrize("M,K,rps,pad", [(256, 3072, 64, 0), (1000, 2240, 333, 16), (77, 64, 10, 0), (130, 4096, 130, 0),
                                         (300, 1024, 1, 8), (513, 2432, 200, 0)])
def test_layernorm_quantize_valid(B, M, K, rps, pad):
    run_case(B, M, K, rps, M + K, pad)


def test_flux_sized_input_sampled(B):
    # FLUX hidden size, one full 4608-token sample group of 8: every row through the kernel, the
    # oracle on a sample of rows (whole 128-row tiles at both ends plus scattered rows)
    M, K, rps = 36864, 3072, 4608
    g = torch.Generator(device="cuda").manual_seed(3)
    x = workloads.make_activation("student_t", M, K, g, "cuda")
    scale = (torch.randn(8, K, generator=g, device="cuda") * 0.3).to(torch.bfloat16)
    shift = (torch.randn(8, K, generator=g, device="cuda") * 0.2).to(torch.bfloat16)
    ts = torch.tensor([0.004], dtype=torch.float32, device="cuda")
    q, sf = B.nvfp4_layernorm_quantize(x, scale, shift, rps, ts)
    rows = np.unique(np.concatenate([np.arange(128), np.arange(M - 128, M), np.random.default_rng(0).integers(0, M, 256)]))
    rows_t = torch.from_numpy(rows).cuda()
    xb = bits_of(x[rows_t])
    # the oracle takes whole sample groups: evaluate each sampled row with its own sample's modulation
    Y = np.empty((rows.size, K))
    for s_idx in range(8):
        sel = (rows // rps) == s_idx
        if sel.any():
            Y[sel] = oracle.layernorm_modulate(xb[sel], bits_of(scale[s_idx:s_idx + 1]), bits_of(shift[s_idx:s_idx + 1]),
                                               10 ** 9)
    q_star, sf_star = oracle.quantize(oracle.round_bf16(Y), 0.004)
    sf_rm = unswizzle_rows(sf.cpu().numpy(), rows, K)
    codes, codes_star = nibbles(q[rows_t].cpu().numpy()), nibbles(q_star)
    assert (sf_rm == sf_star).mean() >= 0.995 and (codes == codes_star).mean() >= 0.99
    assert np.abs(sf_rm.astype(np.int32) - sf_star.astype(np.int32)).max() <= 1


def test_rejects_bad_arguments(B):
    x = torch.zeros((4, 96), dtype=torch.bfloat16, device="cuda")
    m = torch.zeros((1, 96), dtype=torch.bfloat16, device="cuda")
    t = torch.ones(1, dtype=torch.float32, device="cuda")
    with pytest.raises(B.SolError):
        B.nvfp4_layernorm_quantize(x, m, m, 4, t)        # K % 64
