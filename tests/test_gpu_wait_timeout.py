"""The bounded-wait path of the GEMM kernels, run for real: a wait that nothing satisfies expires
after a short limit, the kernel leaves through its normal teardown, the host reads SOL_ERR_TIMEOUT
with the code of the wait that gave up, and the next ordinary call works.  No trap, no fault, no
unbounded spin: the load-issuing warps simply issue nothing while the test hook is on."""
import pytest
import torch

from paper_2604_06916_b200 import workloads

pytestmark = pytest.mark.gpu

SOL_ERR_TIMEOUT = 7
# wait sites (high byte of the status word): 0x1 / 0x8 producers on `empty`, 0x3 MMA on `full`,
# 0x4 epilogue on `acc_full`, 0x5 MMA on `sf_ready`, 0x6 / 0x7 scale-copy warps
CONSUMER_SITES = {0x3, 0x4, 0x5, 0x6, 0x7}


@pytest.fixture(scope="module")
def B():
    from paper_2604_06916_b200 import binding
    binding.lib()
    return binding


@pytest.mark.parametrize("which", ["nvfp4", "bf16"])
def test_wait_that_runs_out_is_reported_and_the_context_stays_usable(B, which):
    X, W, bias = workloads.make_layer(workloads.CONFIG_SANA, 1, "cuda", M=1024)
    wq, wsf, wts = B.nvfp4_quantize_weight(W)
    xts = B.sol_amax_bf16(X)
    xq, xsf = B.nvfp4_quantize(X, xts)

    def run(out):
        if which == "nvfp4":
            return B.nvfp4_linear(xq, xsf, xts, wq, wsf, wts, bias, out=out)
        return B.bf16_linear(X, W, bias, out=out)

    want = run(None)
    B.sol_last_device_status()
    sentinel = torch.full_like(want, 3.0)
    try:
        B.sol_set_wait_limit_cycles(1_000_000)      # about half a millisecond
        B.sol_test_hold_loads(True)
        run(sentinel)
        with pytest.raises(B.SolError) as info:
            B.sol_last_device_status()
    finally:
        B.sol_test_hold_loads(False)
        B.sol_set_wait_limit_cycles(0)
    assert info.value.code == SOL_ERR_TIMEOUT
    assert (info.value.detail >> 8) in CONSUMER_SITES, hex(info.value.detail)
    assert torch.all(sentinel == 3.0)               # the held launch wrote nothing
    B.sol_last_device_status()                      # the word was cleared by the read
    again = run(None)
    B.sol_last_device_status()
    assert torch.equal(again, want)
