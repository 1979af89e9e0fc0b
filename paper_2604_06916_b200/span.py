"""SM cycles and SM clock of the NVFP4 pair GEMM, measured by the kernel itself.

    python -m paper_2604_06916_b200.span [--shape M K N]... [--launches 200] [--zero]

Builds a second copy of the library with -DSOL_SPAN (the product kernel plus one `clock64` and one
`globaltimer` read at both ends of CTA 0), loads it instead of the product library, runs `launches`
back-to-back `nvfp4_linear` calls per shape and prints, for the last launch, the cycles and nanoseconds of
CTA 0: their ratio is the clock the kernel ran at under the board's power cap, and cycles per k-tile
against the tensor pipe's 512 (four 256 x 256 x 64 pair MMAs of 128 cycles) is how far the kernel is from
the pipe, independent of that clock.  A diagnostic: nothing in the library, the tests or bench.py uses it.
"""
from __future__ import annotations

import argparse
import ctypes
import os
import subprocess
import sys

from . import build as _build

SPAN_LIB = os.path.join(_build.HERE, "libsol_nvfp4_span.so")
FLUX_SHAPES = [(36864, 15360, 3072), (36864, 3072, 21504), (36864, 3072, 9216), (36864, 3072, 3072)]


def build_span_library() -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-DSOL_SPAN",
           "-Xcompiler", "-fPIC", "-shared", "-o", SPAN_LIB]
    cmd += [os.path.join(_build.CSRC, s) for s in _build.SOURCES]
    subprocess.run(cmd, check=True)
    return SPAN_LIB


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--shape", type=int, nargs=3, action="append", metavar=("M", "K", "N"))
    ap.add_argument("--launches", type=int, default=200)
    ap.add_argument("--zero", action="store_true", help="all-zero activations (lowest power draw)")
    args = ap.parse_args(argv)

    os.environ["SOL_NVFP4_LIB"] = build_span_library()   # before the binding resolves its library path
    import torch
    from . import binding as B

    pairs = torch.cuda.get_device_properties(0).multi_processor_count // 2
    for (M, K, N) in (args.shape or FLUX_SHAPES):
        g = torch.Generator(device="cuda").manual_seed(1)
        X = torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16)
        W = (torch.randn(N, K, generator=g, device="cuda") * K ** -0.5).to(torch.bfloat16)
        if args.zero:
            X.zero_()
        wq, wsf, wts = B.nvfp4_quantize_weight(W)
        xts = B.sol_amax_bf16(X)
        xq, xsf = B.nvfp4_quantize(X, xts)
        Y = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
        for _ in range(10):
            B.nvfp4_linear(xq, xsf, xts, wq, wsf, wts, None, out=Y)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.launches):
            B.nvfp4_linear(xq, xsf, xts, wq, wsf, wts, None, out=Y)
        e1.record()
        torch.cuda.synchronize()
        B.sol_last_device_status()
        ms = e0.elapsed_time(e1) / args.launches
        span = (ctypes.c_longlong * 2)()
        if B.lib().sol_debug_span(span) != 0:
            raise RuntimeError("sol_debug_span failed")
        cycles, ns = span[0], span[1]
        tiles = -(-M // 256) * -(-N // 256)
        mine = -(-tiles // pairs)                       # tiles of the first CTA pair
        k_tiles = -(-K // 256)
        print(f"M={M} K={K} N={N}: {ms * 1e3:.1f} us per launch ({2.0 * M * N * K / ms / 1e9:.0f} TFLOP/s); "
              f"CTA 0: {cycles} cycles in {ns / 1e3:.1f} us = {cycles / ns * 1e3:.0f} MHz; "
              f"{cycles / (mine * k_tiles):.0f} cycles per k-tile over {mine} tiles x {k_tiles} k-tiles (pipe: 512)")
        del X, W, Y, xq, xsf
    return 0


if __name__ == "__main__":
    sys.exit(main())
