"""GPU parity: adapter merge + weight re-quantization against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_06916_b200 import binding as B
from paper_2604_06916_b200 import workloads

from tests.helpers import bits_of, from_bits, unswizzle_rows

pytestmark = pytest.mark.gpu


def run_case(W, A, Bm, scaling, layout=B.SF_ROW_MAJOR):
    merged, q, sf, ts = B.nvfp4_requantize_lora(W, A, Bm, scaling, layout=layout)
    torch.cuda.synchronize()
    B.sol_last_device_status()
    want_merged, want_q, want_sf, want_T = oracle.requantize_lora(bits_of(W), bits_of(A), bits_of(Bm), scaling)
    assert np.array_equal(bits_of(merged), want_merged)
    assert np.float32(ts.item()) == want_T
    assert np.array_equal(q.cpu().numpy(), want_q)
    N, K = W.shape
    if layout == B.SF_ROW_MAJOR:
        assert np.array_equal(sf.cpu().numpy().reshape(N, K // 16), want_sf)
    else:
        got = unswizzle_rows(sf.cpu().numpy().ravel(), np.arange(N), K)
        assert np.array_equal(got, want_sf)
        assert np.array_equal(sf.cpu().numpy().ravel(), oracle.sf_swizzle(want_sf, K).ravel())


@pytest.mark.parametrize("N,K,r", [
    (64, 256, 32),        # exactly one tile
    (200, 1056, 32),      # ragged rows and columns, several tiles
    (8, 32, 1),           # smallest shape, rank 1
    (136, 608, 64),       # largest rank
    (1024, 2240, 32),     # a SANA-sized projection (K = 2240 is not a multiple of 256)
    (72, 320, 7),         # odd rank
])
@pytest.mark.parametrize("layout", [B.SF_ROW_MAJOR, B.SF_SWIZZLED_128x4])
def test_merge_and_requantize_matches_oracle(N, K, r, layout):
    g = torch.Generator(device="cuda").manual_seed(N * 7 + K + r)
    W = (torch.randn(N, K, generator=g, device="cuda") * K ** -0.5).to(torch.bfloat16)
    A, Bm = workloads.make_lora(N, K, seed=r, device="cuda", rank=r)
    run_case(W, A, Bm, workloads.LORA_ALPHA / workloads.LORA_RANK, layout)


def test_strided_inputs_and_scaling_not_a_power_of_two():
    g = torch.Generator(device="cuda").manual_seed(3)
    N, K, r = 96, 512, 32
    Wbig = (torch.randn(N, K + 64, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    Abig = (torch.randn(r, K + 32, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    Bbig = (torch.randn(N, r + 5, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    run_case(Wbig[:, :K], Abig[:, :K], Bbig[:, :r], 0.75)


def test_cancellation_follows_the_fixed_order():
    # the hand-worked case of the CPU pins: 2^24 + 1 - 2^24 summed in rank order gives 0
    N, K = 8, 32
    W = torch.full((N, K), 0.5, dtype=torch.bfloat16, device="cuda")
    A = torch.zeros((3, K), dtype=torch.bfloat16, device="cuda")
    A[0, :], A[1, :], A[2, :] = 4096.0, 1.0, 4096.0
    Bm = torch.zeros((N, 3), dtype=torch.bfloat16, device="cuda")
    Bm[:, 0], Bm[:, 1], Bm[:, 2] = 4096.0, 1.0, -4096.0
    merged, _, _, _ = B.nvfp4_requantize_lora(W, A, Bm, 2.0)
    assert torch.all(merged.float() == 0.5)
    merged, _, _, _ = B.nvfp4_requantize_lora(W, A.flip(0).contiguous(), Bm.flip(1).contiguous(), 2.0)
    assert torch.all(merged.float() == 2.5)
    run_case(W, A, Bm, 2.0)


def test_zero_adapter_equals_plain_weight_quantizer():
    g = torch.Generator(device="cuda").manual_seed(9)
    N, K = 256, 768
    W = (torch.randn(N, K, generator=g, device="cuda") * 0.03).to(torch.bfloat16)
    A, _ = workloads.make_lora(N, K, seed=1, device="cuda")
    Z = torch.zeros((N, 32), dtype=torch.bfloat16, device="cuda")
    merged, q, sf, ts = B.nvfp4_requantize_lora(W, A, Z, 2.0)
    q0, sf0, ts0 = B.nvfp4_quantize_weight(W)
    assert torch.equal(merged, W) and torch.equal(q, q0) and torch.equal(sf, sf0) and torch.equal(ts, ts0)


def test_full_size_flux_projection_sampled_rows():
    # a FLUX attention projection (3072 x 3072, rank 32) in the launch configuration the benchmark
    # times; the oracle recomputes a sample of rows, T is checked through the full-tensor amax
    N = K = 3072
    _, W, _ = workloads.make_layer(workloads.CONFIG_FLUX, 1, "cuda", M=128)
    A, Bm = workloads.make_lora(N, K, seed=1, device="cuda")
    merged, q, sf, ts = B.nvfp4_requantize_lora(W, A, Bm, 2.0)
    torch.cuda.synchronize()
    rows = np.unique(np.concatenate([np.arange(0, 64), np.arange(N - 64, N),
                                     np.random.default_rng(0).integers(0, N, 192)]))
    wb, ab, bb = bits_of(W), bits_of(A), bits_of(Bm)
    want = oracle.lora_merge(wb[rows], ab, bb[rows], 2.0)
    got = bits_of(merged)
    assert np.array_equal(got[rows], want)
    T = np.float32(ts.item())
    amax = np.float32(np.abs(oracle.bits_to_f64(got)).max())
    assert T == np.float32(amax / np.float32(2688.0))
    want_q, want_sf = oracle.quantize(want, T)
    assert np.array_equal(q.cpu().numpy()[rows], want_q)
    assert np.array_equal(unswizzle_rows(sf.cpu().numpy().ravel(), rows, K), want_sf)


def test_rejects_bad_arguments():
    W = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    A = torch.zeros((65, 64), dtype=torch.bfloat16, device="cuda")
    Bm = torch.zeros((64, 65), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.SolError):
        B.nvfp4_requantize_lora(W, A, Bm, 2.0)  # rank above the supported maximum


@pytest.mark.parametrize("group", [1, 2, 4, 8])
def test_batch_entry_equals_single_calls(group):
    N, K, r = 192, 640, 32
    items = []
    for i in range(5):
        g = torch.Generator(device="cuda").manual_seed(100 + i)
        W = (torch.randn(N, K, generator=g, device="cuda") * 0.04).to(torch.bfloat16)
        A, Bm = workloads.make_lora(N, K, seed=i, device="cuda")
        items.append((W, A, Bm))
    plan = B.LoraRefreshPlan(items, 2.0, group=group)
    outs = plan.run()
    torch.cuda.synchronize()
    for (W, A, Bm), (q, sf, ts) in zip(items, outs):
        merged1, q1, sf1, ts1 = B.nvfp4_requantize_lora(W, A, Bm, 2.0)
        assert torch.equal(q, q1) and torch.equal(sf, sf1) and torch.equal(ts[:1], ts1)
    # second run on the same buffers gives the same result (no state carried between calls)
    keep = [(q.clone(), sf.clone(), ts.clone()) for q, sf, ts in outs]
    plan.run()
    torch.cuda.synchronize()
    for (q, sf, ts), (q0, sf0, ts0) in zip(plan.outputs, keep):
        assert torch.equal(q, q0) and torch.equal(sf, sf0) and torch.equal(ts, ts0)
