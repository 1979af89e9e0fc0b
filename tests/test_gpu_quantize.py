"""GPU parity: amax and NVFP4 quantizer vs the CPU oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_06916_b200 import workloads
from tests.helpers import bits_of, from_bits, swizzled_offsets

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06916_b200 import binding
    binding.lib()
    return binding


def compare_quantized(B, x: torch.Tensor, what: str):
    """Quantize x (a view with any row pitch) on the GPU in both scale layouts; compare with the oracle."""
    xb = bits_of(x)
    M, K = xb.shape
    T_gpu = B.sol_amax_bf16(x)
    T = oracle.tensor_scale(xb)
    assert T_gpu.cpu().numpy().view(np.uint32)[0] == np.float32(T).view(np.uint32), what
    q_ref, sf_ref = oracle.quantize(xb, T)
    q, sf = B.nvfp4_quantize(x, T_gpu, B.SF_ROW_MAJOR)
    q2, sf2 = B.nvfp4_quantize(x, T_gpu, B.SF_SWIZZLED_128x4)
    torch.cuda.synchronize()
    q, sf, q2, sf2 = q.cpu().numpy(), sf.cpu().numpy(), q2.cpu().numpy(), sf2.cpu().numpy()
    nbad = int(np.count_nonzero(q != q_ref))
    assert nbad == 0, f"{what}: {nbad} packed bytes differ; first at {np.argwhere(q != q_ref)[0]}"
    assert np.array_equal(sf.reshape(M, K // 16), sf_ref), what
    assert np.array_equal(q2, q_ref), what
    assert np.array_equal(sf2, oracle.sf_swizzle(sf_ref, K)), f"{what}: swizzled scales or zero padding differ"
    return T


def test_config1_single_layer_full(B):
    X, W, _ = workloads.make_layer(workloads.CONFIG_SINGLE, 0, "cuda")
    compare_quantized(B, X, "config1 X")
    compare_quantized(B, W, "config1 W")


@pytest.mark.parametrize("M,K,pad", [(1, 32, 0), (130, 160, 0), (257, 2240, 8), (40, 5600, 64), (300, 96, 32)])
def test_ragged_shapes_and_row_pitch(B, M, K, pad):
    gen = torch.Generator(device="cuda").manual_seed(100 + M)
    full = workloads.make_activation("student_t", M, K + pad, gen, "cuda")
    compare_quantized(B, full[:, :K], f"M={M} K={K} pitch={K + pad}")


def test_special_values_signed_zero_ties_saturation(B):
    vals = [6, 3, 1.5, -0.75, 0.25, 5, 2.5, -6, 0.1, 0, -0.0, 0, 0, 0, 0, 0]   # hand-worked block
    vals += [0.0, -0.0] * 8                                                    # zero block keeps sign bits
    vals += [6.25, -1.75, 1.25, 3.5, -3.5, 0.75, 5.0, -5.0] + [0.0] * 8        # ties, saturating max
    vals += [2.0 ** -20] * 16                                                  # underflowing block scale
    x = torch.tensor([vals, [-v for v in vals]], dtype=torch.float32).to(torch.bfloat16).cuda()
    one = torch.ones(1, dtype=torch.float32, device="cuda")
    xb = bits_of(x)
    q_ref, sf_ref = oracle.quantize(xb, 1.0)
    q, sf = B.nvfp4_quantize(x, one, B.SF_ROW_MAJOR)
    assert np.array_equal(q.cpu().numpy(), q_ref)
    assert np.array_equal(sf.cpu().numpy().reshape(2, -1), sf_ref)
    assert list(q_ref[0, :8]) == [0x57, 0xA3, 0x60, 0xF4, 0x00, 0x08, 0x00, 0x00]
    zero = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    assert B.sol_amax_bf16(zero).item() == 1.0


def test_vectorised_offset_helper_matches_oracle_rule():
    K = 2240
    offs = swizzled_offsets(np.array([0, 31, 32, 127, 128, 300]), K)
    for i, r in enumerate([0, 31, 32, 127, 128, 300]):
        for b in (0, 1, 3, 4, 139):
            assert offs[i, b] == oracle.sf_swizzled_offset(r, b, K)


@pytest.mark.parametrize("cfg_name,index", [
    ("sana_1p6b_g16", 0), ("sana_1p6b_g16", 3), ("sd35_large_g8", 0), ("sd35_large_g8", 3),
    ("flux1_12b_g8", 0), ("flux1_12b_g8", 5),
])
def test_full_size_activation_tensors(B, cfg_name, index):
    cfg = workloads.CONFIGS[cfg_name]
    X, _, _ = workloads.make_layer(cfg, index, "cuda")
    compare_quantized(B, X, f"{cfg_name}/{cfg.layers[index].name}")


def test_weight_quantizer_entry(B):
    cfg = workloads.CONFIG_SANA
    _, W, _ = workloads.make_layer(cfg, 3, "cuda", M=128)
    q, sf, ts = B.nvfp4_quantize_weight(W)
    wb = bits_of(W)
    T = oracle.tensor_scale(wb)
    assert ts.cpu().numpy().view(np.uint32)[0] == np.float32(T).view(np.uint32)
    q_ref, sf_ref = oracle.quantize(wb, T)
    assert np.array_equal(q.cpu().numpy(), q_ref)
    assert np.array_equal(sf.cpu().numpy(), oracle.sf_swizzle(sf_ref, W.shape[1]))


def test_deterministic_run_to_run(B):
    X, _, _ = workloads.make_layer(workloads.CONFIG_SANA, 0, "cuda", M=4096)
    T = B.sol_amax_bf16(X)
    a = B.nvfp4_quantize(X, T)
    b = B.nvfp4_quantize(X, T)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
