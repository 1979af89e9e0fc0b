"""The allocation-free fused entry (scratch in a fixed device array inside the library) must give
exactly what the workspace-taking entry gives, call after call.

Kept in a file that sorts last so that a run stopping at the first failure has already run the
rest of the suite.  It must pass alone in a fresh process as well as after the other tests.
"""
import pytest
import torch

from paper_2604_06916_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06916_b200 import binding
    binding.lib()
    return binding


def test_static_scratch_entry_matches_workspace_entry_twice_in_a_row(B):
    cfg = workloads.CONFIG_SANA
    outs = []
    for index, rows in ((1, 3000), (0, 1111)):   # two different problems, back to back, same array
        X, W, bias = workloads.make_layer(cfg, index, "cuda", M=rows)
        wq, wsf, wts = B.nvfp4_quantize_weight(W)
        want = B.nvfp4_quantize_linear(X, wq, wsf, wts, bias)
        got = torch.full_like(want, float("nan"))
        B.nvfp4_quantize_linear_static(X, wq, wsf, wts, bias, out=got)
        B.sol_last_device_status()
        assert torch.equal(got, want)             # same kernels, same inputs: bit-identical BF16
        outs.append((X, wq, wsf, wts, bias, want))
    # and once more on the first problem: old contents of the shared array must not leak in
    X, wq, wsf, wts, bias, want = outs[0]
    assert torch.equal(B.nvfp4_quantize_linear_static(X, wq, wsf, wts, bias), want)


def test_static_scratch_entry_rejects_oversized_problems(B):
    limit = B.static_scratch_bytes()
    assert limit == 64 << 20
    M, K, N = 65536, 4096, 64                      # needs ~151 MB of scratch
    assert B.linear_workspace_bytes(M, N, K) > limit
    x = torch.empty((8, K), dtype=torch.bfloat16, device="cuda")  # never read: the call must refuse first
    wq = torch.empty((N, K // 2), dtype=torch.uint8, device="cuda")
    wsf = torch.empty(B.scale_bytes(N, K), dtype=torch.uint8, device="cuda")
    wts = torch.ones(1, dtype=torch.float32, device="cuda")
    y = torch.empty((8, N), dtype=torch.bfloat16, device="cuda")
    code = B.lib().nvfp4_quantize_linear_static(x.data_ptr(), K, wq.data_ptr(), wsf.data_ptr(), wts.data_ptr(), None,
                                                y.data_ptr(), M, N, K, N, None)
    assert B.status_string(code) == "SOL_ERR_WORKSPACE_TOO_SMALL"
