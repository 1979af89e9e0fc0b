"""CPU-only checks of the boundary: the shared library loads and exports every symbol the header
declares, size queries, argument validation (no kernel is launched on an error), and the
multi-rank timing aggregation on a world-size-2 gloo group."""
import ctypes
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "sol_nvfp4.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2604_06916_b200 import build

    path = build.build()
    from paper_2604_06916_b200 import binding

    return binding.lib()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b([a-z_0-9]+)\s*\(", text)) - {"defined"})


def test_library_exports_every_declared_symbol(lib):
    from paper_2604_06916_b200 import binding

    names = declared_functions()
    assert set(binding.EXPORTS) == set(names)
    raw = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n


def test_status_strings(lib):
    from paper_2604_06916_b200 import binding as B

    assert B.status_string(0) == "SOL_OK"
    assert B.status_string(4) == "SOL_ERR_WORKSPACE_TOO_SMALL"
    assert B.status_string(7) == "SOL_ERR_TIMEOUT"
    assert B.status_string(99) == "SOL_ERR_UNKNOWN"


def test_size_queries(lib):
    from paper_2604_06916_b200 import binding as B

    assert B.data_bytes(256, 512) == 256 * 256
    assert B.scale_bytes(256, 512, B.SF_ROW_MAJOR) == 256 * 32
    assert B.scale_bytes(256, 512, B.SF_SWIZZLED_128x4) == 2 * 8 * 512
    assert B.scale_bytes(130, 160, B.SF_SWIZZLED_128x4) == 2 * 3 * 512       # padded rows and k chunks
    assert B.scale_bytes(40, 5600, B.SF_SWIZZLED_128x4) == 1 * 88 * 512
    assert B.data_bytes(16, 24) == 0 and B.scale_bytes(0, 64) == 0            # K % 32, rows > 0
    ws = B.linear_workspace_bytes(36864, 3072, 3072)
    assert ws >= B.data_bytes(36864, 3072) + B.scale_bytes(36864, 3072) + 4 and ws % 256 == 0
    assert B.static_scratch_bytes() == 64 << 20


def test_argument_validation_happens_before_any_cuda_call(lib):
    """Bad arguments are refused on the host; this box has no GPU, so reaching CUDA would fail differently."""
    L = lib
    buf = ctypes.create_string_buffer(4096)
    p = (ctypes.addressof(buf) + 255) & ~255   # aligned fake pointer, never dereferenced
    NULLP, SHAPE, ALIGN, WS, LAYOUT = 1, 2, 3, 4, 8
    assert L.sol_amax_bf16(None, 4, 64, 64, p, None) == NULLP
    assert L.sol_amax_bf16(p, 4, 48, 48, p, None) == SHAPE                     # K % 32
    assert L.sol_amax_bf16(p, 4, 64, 32, p, None) == SHAPE                     # ld < K
    assert L.sol_amax_bf16(p + 2, 4, 64, 64, p, None) == ALIGN
    assert L.nvfp4_quantize(p, 4, 64, 64, None, p, p, 1, None) == NULLP
    assert L.nvfp4_quantize(p, 4, 64, 64, p, p, p, 5, None) == LAYOUT
    assert L.nvfp4_quantize(p, 0, 64, 64, p, p, p, 1, None) == SHAPE
    assert L.nvfp4_quantize(p, 4, 64, 68, p, p, p, 1, None) == ALIGN           # pitch not a multiple of 8
    assert L.nvfp4_quantize_weight(p, 4, 64, 64, p, p, None, 1, None) == NULLP
    assert L.nvfp4_linear(p, p, p, p, p, p, None, None, 4, 8, 64, 8, None) == NULLP
    assert L.nvfp4_linear(p, p, p, p, p, p, None, p, 4, 12, 64, 16, None) == SHAPE   # N % 8
    assert L.nvfp4_linear(p, p, p, p, p, p, None, p, 4, 8, 64, 4, None) == SHAPE     # ldy < N
    assert L.nvfp4_linear(p, p, p, p, p, p, p + 8, p, 4, 8, 64, 8, None) == ALIGN    # bias alignment
    assert L.bf16_linear(p, p, None, p, 4, 8, 64, 32, 64, 8, None) == SHAPE          # ldx < K
    assert L.bf16_linear(None, p, None, p, 4, 8, 64, 64, 64, 8, None) == NULLP
    assert L.nvfp4_quantize_linear(p, 64, p, p, p, None, p, 4, 8, 64, 8, None, 0, None) == NULLP
    assert L.nvfp4_quantize_linear(p, 64, p, p, p, None, p, 4, 8, 64, 8, p, 16, None) == WS
    assert L.nvfp4_quantize_linear(p, 64, p, p, p, None, p, 4, 8, 64, 8, p + 16, 1 << 20, None) == ALIGN
    assert L.nvfp4_quantize_linear_static(p, 4096, p, p, p, None, p, 1 << 20, 8, 4096, 8, None) == WS
    assert L.nvfp4_quantize_linear_static(None, 64, p, p, p, None, p, 4, 8, 64, 8, None) == NULLP
    # weight refresh
    assert L.nvfp4_requantize_lora(p, 64, p, 64, p, 32, 8, 64, 32, 2.0, None, p, p, p, 1, None) == NULLP
    assert L.nvfp4_requantize_lora(p, 64, p, 64, p, 32, 8, 64, 65, 2.0, p, p, p, p, 1, None) == SHAPE   # rank > 64
    assert L.nvfp4_requantize_lora(p, 64, p, 64, p, 16, 8, 64, 32, 2.0, p, p, p, p, 1, None) == SHAPE   # ldb < r
    assert L.nvfp4_requantize_lora(p, 64, p, 64, p + 1, 32, 8, 64, 32, 2.0, p, p, p, p, 1, None) == ALIGN
    assert L.nvfp4_requantize_lora(p, 64, p, 64, p, 32, 8, 64, 32, 2.0, p, p, p, p, 7, None) == LAYOUT
    lst = (ctypes.c_void_p * 2)(p, p)
    bad = (ctypes.c_void_p * 2)(p, None)
    assert L.nvfp4_requantize_lora_batch(0, None, None, None, None, None, None, 8, 64, 32, 2.0, p, 1, 1, None) == 0
    assert L.nvfp4_requantize_lora_batch(2, lst, lst, lst, lst, lst, None, 8, 64, 32, 2.0, p, 1, 1, None) == NULLP
    assert L.nvfp4_requantize_lora_batch(2, lst, bad, lst, lst, lst, lst, 8, 64, 32, 2.0, p, 1, 1, None) == NULLP
    assert L.nvfp4_requantize_lora_batch(2, lst, lst, lst, lst, lst, lst, 8, 64, 32, 2.0, p, 0, 1, None) == SHAPE
    assert L.nvfp4_requantize_lora_batch(-1, lst, lst, lst, lst, lst, lst, 8, 64, 32, 2.0, p, 1, 1, None) == SHAPE
    # stage-1 selection and rank metrics
    assert L.solrl_select_contrastive(None, None, 2, 8, 4, p, None, None, None) == NULLP
    assert L.solrl_select_contrastive(p, None, 2, 8, 4, p, p, None, None) == NULLP      # seeds_out without seeds
    assert L.solrl_select_contrastive(p, None, 2, 8, 5, p, None, None, None) == SHAPE   # odd K
    assert L.solrl_select_contrastive(p, None, 2, 8, 10, p, None, None, None) == SHAPE  # K > N
    assert L.solrl_select_contrastive(p, None, 2, 5000, 4, p, None, None, None) == SHAPE
    assert L.solrl_select_contrastive(p + 2, None, 2, 8, 4, p, None, None, None) == ALIGN
    assert L.solrl_rank_consistency(p, None, 2, 8, 4, p, None, None) == NULLP
    assert L.solrl_rank_consistency(p, p, 2, 1, 1, p, None, None) == SHAPE
    assert L.solrl_rank_consistency(p, p, 2, 8, 9, p, None, None) == SHAPE
    assert L.solrl_rank_consistency(p, p, 2, 8, 4, p + 4, None, None) == ALIGN
    # split output and quantize-into-slice
    assert L.nvfp4_linear_split_out(p, p, p, p, p, p, None, None, 256, 256, 0, p, p, p, 256, 0, None, 4, 512, 64, None) == NULLP
    assert L.nvfp4_linear_split_out(p, p, p, p, p, p, None, p, 256, 128, 0, p, p, p, 256, 0, None, 4, 512, 64, None) == SHAPE   # n_split % 256
    assert L.nvfp4_linear_split_out(p, p, p, p, p, p, None, p, 256, 256, 0, p, p, p, 256, 64, None, 4, 512, 64, None) == SHAPE  # part does not fit
    assert L.nvfp4_linear_split_out(p, p, p, p, p, p, None, p, 256, 256, 0, p, p, p, 320, 32, None, 4, 512, 64, None) == SHAPE  # dest_col0 % 64
    assert L.nvfp4_linear_split_out(p, p, p, p, p, p, None, p, 256, 256, 0, p, p + 8, p, 256, 0, None, 4, 512, 64, None) == ALIGN
    assert L.nvfp4_quantize_into(p, 4, 64, 64, p, None, p, 128, 0, None) == NULLP
    assert L.nvfp4_quantize_into(p, 4, 96, 96, p, p, p, 192, 0, None) == SHAPE     # K % 64
    assert L.nvfp4_quantize_into(p, 4, 64, 64, p, p, p, 128, 128, None) == SHAPE   # past the end
    assert L.nvfp4_quantize_into(p, 4, 64, 64, p, p + 4, p, 128, 0, None) == ALIGN
    # delayed tensor scale
    assert L.nvfp4_quantize_linear_delayed(p, 64, p, p, p, None, p, 4, 8, 64, 8, None, p, 1 << 20, None) == NULLP
    assert L.nvfp4_quantize_linear_delayed(p, 64, p, p, p, None, p, 4, 8, 64, 8, p + 4, p, 1 << 20, None) == ALIGN
    assert L.nvfp4_quantize_linear_delayed(p, 64, p, p, p, None, p, 4, 8, 64, 8, p, p, 16, None) == WS
    assert L.sol_roll_tensor_scale(None, None) == NULLP
    # layer norm fused with the quantizer
    assert L.nvfp4_layernorm_quantize(p, 4, 64, 64, p, None, 4, 1e-6, p, p, p, None, None) == NULLP
    assert L.nvfp4_layernorm_quantize(p, 4, 96, 96, p, p, 4, 1e-6, p, p, p, None, None) == SHAPE      # K % 64
    assert L.nvfp4_layernorm_quantize(p, 4, 8192, 8192, p, p, 4, 1e-6, p, p, p, None, None) == SHAPE  # K > 4096
    assert L.nvfp4_layernorm_quantize(p, 4, 64, 64, p, p, 0, 1e-6, p, p, p, None, None) == SHAPE
    assert L.nvfp4_layernorm_quantize(p, 4, 64, 64, p + 8, p, 4, 1e-6, p, p, p, None, None) == ALIGN
    # attention
    assert L.sol_attention_bf16(p, p, None, p, 1, 4, 4, 1, 128, 128, 128, 128, 128, None) == NULLP
    assert L.sol_attention_bf16(p, p, p, p, 1, 0, 4, 1, 128, 128, 128, 128, 128, None) == SHAPE
    assert L.sol_attention_bf16(p, p, p, p, 1, 4, 4, 2, 128, 128, 256, 256, 256, None) == SHAPE      # pitch < heads * head_dim
    assert L.sol_attention_bf16(p, p, p, p, 1, 4, 4, 1, 96, 128, 128, 128, 128, None) == SHAPE       # head_dim
    assert L.sol_attention_bf16(p, p, p, p, 70000, 4, 4, 1, 128, 128, 128, 128, 128, None) == SHAPE
    assert L.sol_attention_bf16(p, p, p, p, 1, 4, 4, 1, 128, 132, 128, 128, 128, None) == ALIGN      # pitch % 8
    assert L.sol_attention_bf16(p, p + 8, p, p, 1, 4, 4, 1, 128, 128, 128, 128, 128, None) == ALIGN
    assert L.mxfp4_linear_quantized_out(p, p, p, None, None, 0, p, p, None, 4, 128, 64, None) == NULLP
    assert L.mxfp4_linear_quantized_out(p, p, p, p, None, 0, p, p, None, 4, 192, 64, None) == SHAPE      # N % 128
    assert L.mxfp4_linear_quantized_out(p, p, p, p, None, 0, p + 8, p, None, 4, 128, 64, None) == ALIGN
    assert L.sol_attention_nvfp4_out(p, p, p, 1, 4, 4, 1, 128, 128, 128, 128, None, p, p, 128, 0, None, None) == NULLP
    assert L.sol_attention_nvfp4_out(p, p, p, 1, 4, 4, 1, 128, 128, 128, 128, p, p, p, 96, 0, None, None) == SHAPE     # dest_K % 64
    assert L.sol_attention_nvfp4_out(p, p, p, 1, 4, 4, 1, 128, 128, 128, 128, p, p, p, 128, 64, None, None) == SHAPE   # past the end
    assert L.sol_attention_nvfp4_out(p, p, p, 1, 4, 4, 1, 128, 128, 128, 128, p, p + 8, p, 128, 0, None, None) == ALIGN
    from paper_2604_06916_b200.binding import AttentionStream
    ok = AttentionStream(p, p, p, p, 256, 128, 128, 128, 128)
    assert L.sol_attention_bf16_joint(None, ctypes.byref(ok), 1, 1, 128, None) == NULLP
    assert L.sol_attention_bf16_joint(ctypes.byref(AttentionStream(p, None, p, p, 256, 128, 128, 128, 128)), ctypes.byref(ok), 1, 1, 128, None) == NULLP
    assert L.sol_attention_bf16_joint(ctypes.byref(AttentionStream(p, p, p, p, 200, 128, 128, 128, 128)), ctypes.byref(ok), 1, 1, 128, None) == SHAPE  # first % 256
    assert L.sol_attention_bf16_joint(ctypes.byref(ok), ctypes.byref(AttentionStream(p, p, p, p, 0, 128, 128, 128, 128)), 1, 1, 128, None) == SHAPE
    assert L.sol_attention_bf16_joint(ctypes.byref(ok), ctypes.byref(AttentionStream(p, p, p, p + 8, 5, 128, 128, 128, 128)), 1, 1, 128, None) == ALIGN
    # MXFP4
    assert L.sol_mxfp4_scale_bytes(256, 512, 0) == 256 * 16 and L.sol_mxfp4_scale_bytes(256, 512, 1) == 2 * 4 * 512
    assert L.sol_mxfp4_scale_bytes(130, 160, 1) == 2 * 2 * 512 and L.sol_mxfp4_scale_bytes(4, 48, 1) == 0
    assert L.mxfp4_quantize(None, 4, 64, 64, p, p, 1, None) == NULLP
    assert L.mxfp4_quantize(p, 4, 48, 48, p, p, 1, None) == SHAPE
    assert L.mxfp4_quantize(p, 4, 64, 64, p, p, 3, None) == LAYOUT
    assert L.mxfp4_quantize(p, 4, 64, 68, p, p, 1, None) == ALIGN
    assert L.mxfp4_linear(p, p, p, p, None, None, 4, 8, 64, 8, None) == NULLP
    assert L.mxfp4_linear(p, p, p, p, None, p, 4, 12, 64, 16, None) == SHAPE
    assert L.mxfp4_linear(p, p + 8, p, p, None, p, 4, 8, 64, 8, None) == ALIGN
    # linear with quantized output
    assert L.nvfp4_linear_quantized_out(p, p, p, p, p, p, None, 0, None, p, p, None, 4, 64, 64, None) == NULLP
    assert L.nvfp4_linear_quantized_out(p, p, p, p, p, p, None, 0, p, p, p, None, 4, 96, 64, None) == SHAPE   # N % 64
    assert L.nvfp4_linear_quantized_out(p, p, p, p, p, p, None, 5, p, p, p, None, 4, 64, 64, None) == LAYOUT  # activation
    assert L.nvfp4_linear_quantized_out(p, p, p, p, p, p, None, 0, p, p + 8, p, None, 4, 64, 64, None) == ALIGN


def test_binding_refuses_to_run_without_the_library(tmp_path):
    code = ("import os, sys; sys.path.insert(0, %r); os.environ['SOL_NVFP4_LIB'] = %r\n"
            "from paper_2604_06916_b200 import binding\n"
            "try:\n    binding.lib()\nexcept FileNotFoundError as e:\n    print('refused'); sys.exit(0)\n"
            "sys.exit(1)\n") % (ROOT, str(tmp_path / "missing.so"))
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and "refused" in out.stdout, out.stderr


WORKER = r"""
import os, sys
sys.path.insert(0, %r)
import torch.distributed as dist
from paper_2604_06916_b200 import replicas
rank = int(os.environ["RANK"])
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d", rank=rank, world_size=2)
dist.barrier()
ms, units, world = replicas.aggregate(10.0 + 5.0 * rank, 100.0)
assert (ms, units, world) == (15.0, 200.0, 2), (ms, units, world)
assert abs(replicas.throughput(10.0 + 5.0 * rank, 100.0) - 200.0 / 15e-3) < 1e-6
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_replica_aggregation_world_size_2_gloo():
    import socket

    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER % (ROOT, port)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    for rank, pr in enumerate(procs):
        out, err = pr.communicate(timeout=300)
        assert pr.returncode == 0, err
        assert f"rank {rank} ok" in out


def test_replica_aggregation_without_a_process_group():
    from paper_2604_06916_b200 import replicas

    assert replicas.aggregate(3.0, 7.0) == (3.0, 7.0, 1)


def test_diagnostic_build_of_the_gemm_kernels_compiles(tmp_path):
    """The timeline / drop-one-part switches of the GEMM and attention kernels are compiled in only with
    -DSOL_TUNING; the product never builds them, so this keeps that configuration from rotting."""
    import shutil
    import subprocess

    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        pytest.skip("nvcc not available")
    csrc = os.path.join(ROOT, "paper_2604_06916_b200", "csrc")
    for src in ("gemm_pair_fp4.cu", "gemm_pair.cu", "gemm.cu", "attention.cu"):
        flags = ["-DSOL_TUNING"] + (["-DSOL_SPAN"] if src == "gemm_pair_fp4.cu" else [])  # + cycle / time span of CTA 0
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-std=c++17", *flags, "-c",
                        "-o", str(tmp_path / (src + ".o")), os.path.join(csrc, src)], check=True)


def test_guard_mode_of_the_binding_catches_a_write_past_an_output(monkeypatch):
    """SOL_NVFP4_GUARD=1 puts 4 KB bands round every output the binding allocates and checks them after each
    call; here on host tensors: intact bands pass, one byte behind the buffer is reported."""
    import torch
    from paper_2604_06916_b200 import binding as B

    monkeypatch.setenv("SOL_NVFP4_GUARD", "1")
    t = B._empty((3, 5), torch.bfloat16, "cpu")
    assert t.shape == (3, 5) and t.dtype == torch.bfloat16
    assert t.data_ptr() - B._guard_pending[-1][0].data_ptr() == B.GUARD_BYTES   # keeps the allocation's alignment
    t.fill_(1.0)                                   # writing the whole buffer leaves the bands alone
    B.check_guards("intact")
    u = B._empty(7, torch.uint8, "cpu")
    raw, nbytes = B._guard_pending[-1]
    assert nbytes == 7 and u.numel() == 7
    raw[B.GUARD_BYTES + nbytes] = 0
    with pytest.raises(AssertionError, match="back band"):
        B.check_guards("past the end")
    assert not B._guard_pending                    # forgotten after the check
    monkeypatch.setenv("SOL_NVFP4_GUARD", "0")
    B._empty((2, 2), torch.float32, "cpu")
    assert not B._guard_pending                    # off: plain allocations, nothing to check
