"""GPU parity: BF16 attention (head dimension 128 or 64) through the C ABI against the FP64 oracle.

Tolerance (derived in oracle.attention.attention_tolerance): 2^-8 |O| + 2^-8 max|v| -- output
rounding to BF16, probabilities rounded to BF16 before the product with V, row sum from the
unrounded probabilities.
"""
import numpy as np
import pytest
import torch

from oracle import attention as OA
from paper_2604_06916_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06916_b200 import binding
    binding.lib()
    return binding


def f64(t):
    return t.detach().to(torch.float64).cpu().numpy()


def check(B, q, k, v, rows=None):
    out = B.sol_attention_bf16(q, k, v)
    torch.cuda.synchronize()
    assert B.sol_last_device_status() == 0
    qn, kn, vn = f64(q), f64(k), f64(v)
    ref = OA.attention(qn, kn, vn, rows=rows)
    got = f64(out) if rows is None else f64(out)[:, rows]
    tol = OA.attention_tolerance(ref, vn)
    err = np.abs(got - ref)
    worst = float((err / tol).max())
    assert worst <= 1.0, f"max err/tol {worst:.3f} at {np.unravel_index((err / tol).argmax(), err.shape)}"
    return worst


@pytest.mark.parametrize("batch,seq,heads", [(1, 128, 1), (1, 256, 1), (1, 640, 2), (2, 384, 3)])
def test_whole_tiles(B, batch, seq, heads):
    _, q, k, v = workloads.make_qkv(batch, seq, heads, seq + heads, "cuda")
    check(B, q, k, v)


@pytest.mark.parametrize("seq_q,seq_kv", [(1, 1), (5, 3), (200, 333), (129, 127), (130, 16), (64, 1000)])
def test_ragged_sequences_and_cross_lengths(B, seq_q, seq_kv):
    _, q, _, _ = workloads.make_qkv(2, seq_q, 2, 11, "cuda")
    _, _, k, v = workloads.make_qkv(2, seq_kv, 2, 12, "cuda")
    check(B, q, k, v)


def test_sharp_softmax_moves_the_running_max(B):
    # large scores: the row maximum keeps moving from tile to tile, so O is rescaled in TMEM many times
    _, q, k, v = workloads.make_qkv(1, 1024, 2, 21, "cuda", q_gain=6.0)
    check(B, q, k, v)


def test_dense_tensors_and_output_view(B):
    _, q, k, v = workloads.make_qkv(2, 300, 2, 31, "cuda")
    qd, kd, vd = q.contiguous(), k.contiguous(), v.contiguous()
    want = B.sol_attention_bf16(q, k, v)
    got = B.sol_attention_bf16(qd, kd, vd)
    assert torch.equal(want, got)
    # output into a column slice of a wider buffer; the rest of the buffer is not touched
    wide = torch.full((2, 300, 3 * 256), 7.0, dtype=torch.bfloat16, device="cuda")
    view = wide[:, :, 256:512].unflatten(2, (2, 128))
    B.sol_attention_bf16(q, k, v, out=view)
    torch.cuda.synchronize()
    assert torch.equal(view, want)
    assert torch.all(wide[:, :, :256] == 7.0) and torch.all(wide[:, :, 512:] == 7.0)


def test_value_of_one_gives_one_and_single_hot_key(B):
    _, q, k, v = workloads.make_qkv(1, 512, 1, 41, "cuda")
    ones = torch.ones_like(v)
    assert torch.all(B.sol_attention_bf16(q, k, ones) == 1.0)
    # one key aligned with every query and much longer than the rest: the output is that key's value row
    k2 = k.clone()
    k2[0, 300, 0] = 0
    q2 = torch.zeros_like(q)
    q2[..., 5] = 8.0
    k2[..., 5] = 0
    k2[0, 300, 0, 5] = 64.0
    out = B.sol_attention_bf16(q2, k2, v)
    assert torch.equal(out[0, :, 0], v[0, 300, 0].expand(512, 128))


def test_flux_geometry_sampled_rows(B):
    # the bench's shape: 8 samples x 4608 tokens x 24 heads; the oracle computes 3 query rows per tile position
    _, q, k, v = workloads.make_qkv(8, 4608, 24, 51, "cuda")
    out = B.sol_attention_bf16(q, k, v)
    torch.cuda.synchronize()
    assert B.sol_last_device_status() == 0
    rows = [0, 127, 128, 2303, 4500, 4607]
    for b, h in [(0, 0), (3, 11), (7, 23)]:
        ref = OA.attention(f64(q[b:b + 1, :, h:h + 1]), f64(k[b:b + 1, :, h:h + 1]), f64(v[b:b + 1, :, h:h + 1]), rows=rows)
        got = f64(out[b:b + 1, :, h:h + 1])[:, rows]
        tol = OA.attention_tolerance(ref, f64(v[b:b + 1, :, h:h + 1]))
        assert np.all(np.abs(got - ref) <= tol)
    # and every output against the library routine within a looser screen (both round P to BF16)
    lib = torch.nn.functional.scaled_dot_product_attention(q.transpose(1, 2), k.transpose(1, 2), v.transpose(1, 2))
    d = (out.transpose(1, 2).float() - lib.float()).abs().max().item()
    assert d <= 2.0 ** -6 * 2.5, d


@pytest.mark.parametrize("seq_a,seq_b", [(256, 128), (512, 1000), (256, 1), (768, 4096 - 768 + 37)])
def test_joint_streams(B, seq_a, seq_b):
    # text-like and image-like streams from separate fused projections, attending jointly
    _, qa, ka, va = workloads.make_qkv(2, seq_a, 2, 61, "cuda")
    _, qb, kb, vb = workloads.make_qkv(2, seq_b, 2, 62, "cuda")
    oa, ob = B.sol_attention_bf16_joint((qa, ka, va), (qb, kb, vb))
    torch.cuda.synchronize()
    assert B.sol_last_device_status() == 0
    first, second = tuple(f64(t) for t in (qa, ka, va)), tuple(f64(t) for t in (qb, kb, vb))
    ra, rb = OA.attention_joint(first, second)
    vall = np.concatenate((first[2], second[2]), axis=1)
    for got, ref in ((oa, ra), (ob, rb)):
        tol = OA.attention_tolerance(ref, vall)
        assert np.all(np.abs(f64(got) - ref) <= tol)
    # the same tiles in the same order as one call on the concatenated tensors: bit for bit
    q, k, v = (torch.cat((x, y), dim=1) for x, y in ((qa, qb), (ka, kb), (va, vb)))
    whole = B.sol_attention_bf16(q, k, v)
    assert torch.equal(torch.cat((oa, ob), dim=1), whole)


@pytest.mark.parametrize("batch,seq,heads,dest_cols,col0", [(2, 300, 2, 256, 0), (1, 1024, 3, 1024, 384), (3, 130, 1, 192, 64)])
def test_quantized_output_equals_attention_then_quantizer(B, batch, seq, heads, dest_cols, col0):
    # the fused epilogue must give, bit for bit, what the BF16 kernel followed by the destination-slice
    # quantizer gives (each of which is checked against the oracle on its own); other columns stay untouched
    _, q, k, v = workloads.make_qkv(batch, seq, heads, 71, "cuda")
    M = batch * seq
    o = B.sol_attention_bf16(q, k, v).reshape(M, heads * 128)
    T = B.sol_amax_bf16(o)
    def fresh():
        dq = torch.full((M, dest_cols // 2), 0x5A, dtype=torch.uint8, device="cuda")
        dsf = torch.zeros(B.scale_bytes(M, dest_cols), dtype=torch.uint8, device="cuda")
        return dq, dsf
    want = fresh()
    B.nvfp4_quantize_into(o, T, want, col0)
    got = fresh()
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    B.sol_attention_nvfp4_out(q, k, v, T, got, col0, amax_out=amax)
    torch.cuda.synchronize()
    assert B.sol_last_device_status() == 0
    assert torch.equal(got[0], want[0]) and torch.equal(got[1], want[1])
    assert amax.item() == o.float().abs().max().item()
    # and end to end against the FP64 oracle: every dequantized value within the attention tolerance plus half
    # the widest FP4 step (1 unit of the block scale) of the FP64 output
    from tests.helpers import dequantize_on_device
    cols = heads * 128
    sub_q = got[0][:, col0 // 2:(col0 + cols) // 2].contiguous()
    full = dequantize_on_device(got[0], got[1], M, dest_cols).float()[:, col0:col0 + cols] * T.item()
    ref = OA.attention(f64(q), f64(k), f64(v)).reshape(M, cols)
    step = (full.abs().reshape(M, cols // 16, 16).amax(dim=2, keepdim=True) / 6.0 * 1.0).expand(M, cols // 16, 16).reshape(M, cols)
    tol = OA.attention_tolerance(ref.reshape(batch, seq, heads, 128), f64(v)).reshape(M, cols) + 1.01 * step.cpu().numpy() + 1e-30
    assert sub_q.shape == (M, cols // 2)
    assert np.all(np.abs(full.cpu().numpy().astype(np.float64) - ref) <= tol)


@pytest.mark.parametrize("batch,seq_q,seq_kv,heads", [(1, 128, 128, 1), (2, 640, 640, 3), (2, 200, 333, 2), (1, 1, 1, 1),
                                                       (1, 4096 + 154, 4096 + 154, 2)])
def test_head_dimension_64(B, batch, seq_q, seq_kv, heads):
    # the SD3.5 geometry: 64-wide heads (38 of them there; 4096 image + 154 text tokens at 1024 pixels)
    _, q, _, _ = workloads.make_qkv(batch, seq_q, heads, 81, "cuda", head_dim=64)
    _, _, k, v = workloads.make_qkv(batch, seq_kv, heads, 82, "cuda", head_dim=64)
    if seq_q > 2048:   # the oracle on sampled query rows only
        rows = [0, 127, 128, 255, 256, 2000, 4095, 4096, seq_q - 1]
        check(B, q, k, v, rows=rows)
    else:
        check(B, q, k, v)


def test_head_dimension_64_joint_and_quantized_output(B):
    _, qa, ka, va = workloads.make_qkv(2, 256, 2, 83, "cuda", head_dim=64)
    _, qb, kb, vb = workloads.make_qkv(2, 300, 2, 84, "cuda", head_dim=64)
    oa, ob = B.sol_attention_bf16_joint((qa, ka, va), (qb, kb, vb))
    q, k, v = (torch.cat((x, y), dim=1) for x, y in ((qa, qb), (ka, kb), (va, vb)))
    whole = B.sol_attention_bf16(q, k, v)
    assert torch.equal(torch.cat((oa, ob), dim=1), whole)
    ref = OA.attention(f64(q), f64(k), f64(v))
    assert np.all(np.abs(f64(whole) - ref) <= OA.attention_tolerance(ref, f64(v)))
    # quantizing epilogue against the BF16 kernel followed by the slice quantizer, bit for bit
    M, cols = 2 * 556, 2 * 64
    o = whole.reshape(M, cols)
    T = B.sol_amax_bf16(o)
    def fresh():
        return (torch.full((M, 192 // 2), 0x5A, dtype=torch.uint8, device="cuda"),
                torch.zeros(B.scale_bytes(M, 192), dtype=torch.uint8, device="cuda"))
    want, got = fresh(), fresh()
    B.nvfp4_quantize_into(o, T, want, 64)
    B.sol_attention_nvfp4_out(q, k, v, T, got, 64)
    torch.cuda.synchronize()
    assert B.sol_last_device_status() == 0
    assert torch.equal(got[0], want[0]) and torch.equal(got[1], want[1])
