"""GPU parity on the rollout-scaling sweep (FLUX single-stream pair, seed 4, group sizes 4 / 16 / 64).

These are the only shapes with M up to 294 912: an activation tensor of 9 GB, an output of 6.3e9
elements (more than 2^32) and row tiles past 2^31 / K.  The quantizer is compared bit for bit on
128-row slabs (first, middle, last, and the slabs holding element 2^31 and 2^32 of X), with the tensor
scale taken over the whole tensor; the linears on the first and last 128-row tile in full plus one row
of every other tile, all N columns, within 2^-7 |Y| + 1e-4 rms(row); the fused entry bit for bit
against quantize + GEMM; and nothing may be written past the last row of Y.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_06916_b200 import workloads
from tests.helpers import bits_of, check_linear, sample_rows, unswizzle_rows

pytestmark = pytest.mark.gpu

CANARY_ROWS = 8
CANARY = 0x4D5A  # BF16 bit pattern no output of these layers takes in bulk


@pytest.fixture(scope="module")
def B():
    from paper_2604_06916_b200 import binding
    binding.lib()
    return binding


def oracle_tensor_scale_by_slabs(X: torch.Tensor, slab_rows: int = 16384) -> np.float32:
    """T of the whole tensor from the oracle, one host slab at a time.

    IEEE division by a positive constant is monotone, so the largest per-slab T is the T of the largest
    per-slab amax, i.e. of the tensor's amax.  (A slab of zeros would report T = 1; the Student-t
    activations have none, which is asserted.)
    """
    best = np.float32(0.0)
    for r0 in range(0, X.shape[0], slab_rows):
        xb = bits_of(X[r0:r0 + slab_rows])
        assert np.any(xb & 0x7FFF), "all-zero slab"
        best = max(best, np.float32(oracle.tensor_scale(xb)))
    return best


def slabs_of_interest(M: int, K: int):
    """Row tiles (128 rows) to compare in full: the two ends, the middle, and the tiles that hold
    element 2^31 and element 2^32 of the tensor when it is that large."""
    tiles = M // 128
    picks = {0, tiles // 2, tiles - 1}
    for boundary in (1 << 31, 1 << 32):
        t = (boundary // K) // 128
        if t < tiles:
            picks.update({t, max(0, t - 1)})
    return sorted(picks)


def with_canary(M: int, N: int):
    buf = torch.empty((M + CANARY_ROWS, N), dtype=torch.bfloat16, device="cuda")
    buf[M:].view(torch.int16).fill_(CANARY)
    return buf, buf[:M]


def canary_intact(buf: torch.Tensor, M: int) -> bool:
    return bool((buf[M:].view(torch.int16) == CANARY).all())


@pytest.mark.parametrize("index", [0, 1])            # 3072 -> 21504 and 15360 -> 3072
@pytest.mark.parametrize("group", [4, 16, 64])
def test_sweep_pair_quantizer_slabs_and_sampled_linear_rows(B, group, index):
    cfg = workloads.config_sweep(group)
    layer = cfg.layers[index]
    M, K, N = layer.M, layer.K, layer.N
    assert M % 128 == 0
    X, W, bias = workloads.make_layer(cfg, index, "cuda")

    # ---- tensor scale over the whole tensor, bit for bit
    T = oracle_tensor_scale_by_slabs(X)
    xts = B.sol_amax_bf16(X)
    assert xts.cpu().numpy().view(np.uint32)[0] == np.float32(T).view(np.uint32)

    # ---- quantizer: nibbles and chunked scales of whole 128-row slabs, bit for bit
    xq, xsf = B.nvfp4_quantize(X, xts)
    torch.cuda.synchronize()
    chunk_bytes = (K // 64) * 512
    assert xsf.numel() == (M // 128) * chunk_bytes
    for t in slabs_of_interest(M, K):
        r0 = t * 128
        q_ref, sf_ref = oracle.quantize(bits_of(X[r0:r0 + 128]), T)
        assert np.array_equal(xq[r0:r0 + 128].cpu().numpy(), q_ref), f"G={group} {layer.name}: nibbles of rows {r0}.."
        got_sf = xsf[t * chunk_bytes:(t + 1) * chunk_bytes].cpu().numpy()
        assert np.array_equal(got_sf, oracle.sf_swizzle(sf_ref, K)), f"G={group} {layer.name}: scales of rows {r0}.."

    # ---- linears on sampled rows (both end tiles in full, one row of every other tile), all N columns
    rows = sample_rows(M, seed=100 + index)
    rows_t = torch.from_numpy(rows).cuda()
    wq, wsf, wts = B.nvfp4_quantize_weight(W)
    buf, y = with_canary(M, N)
    B.nvfp4_linear(xq, xsf, xts, wq, wsf, wts, bias, out=y)
    B.sol_last_device_status()
    assert canary_intact(buf, M), "nvfp4_linear wrote past the last row of Y"
    sfw_rm = unswizzle_rows(wsf.cpu().numpy(), np.arange(N), K)
    Y = oracle.nvfp4_linear(xq[rows_t].cpu().numpy(), unswizzle_rows(xsf.cpu().numpy(), rows, K), float(T),
                            wq.cpu().numpy(), sfw_rm, wts.item(), bits_of(bias))
    check_linear(bits_of(y[rows_t]), Y, f"{cfg.name}/{layer.name} nvfp4_linear")
    del Y, xq, xsf

    # ---- fused entry: bit-identical to quantize + GEMM over the whole output
    buf2, y2 = with_canary(M, N)
    B.nvfp4_quantize_linear(X, wq, wsf, wts, bias, out=y2)
    B.sol_last_device_status()
    assert canary_intact(buf2, M), "nvfp4_quantize_linear wrote past the last row of Y"
    same = True
    for r0 in range(0, M, 32768):            # compared in slabs: torch.equal on 6.3e9 elements needs a 6 GB mask
        same = same and torch.equal(y[r0:r0 + 32768], y2[r0:r0 + 32768])
    assert same, "fused entry differs from quantize + GEMM"
    del buf2, y2

    # ---- BF16 stack on the same rows
    buf[M:].view(torch.int16).fill_(CANARY)
    B.bf16_linear(X, W, bias, out=y)
    B.sol_last_device_status()
    assert canary_intact(buf, M), "bf16_linear wrote past the last row of Y"
    Yb = oracle.bf16_linear(bits_of(X[rows_t]), bits_of(W), bits_of(bias))
    check_linear(bits_of(y[rows_t]), Yb, f"{cfg.name}/{layer.name} bf16_linear")
