"""B200-native NVFP4 (W4A4) linear layers: quantizer, block-scaled FP4 GEMM, BF16 GEMM.

The compute lives in a C-ABI CUDA library (``csrc/``, declared in ``include/sol_nvfp4.h``);
``binding`` marshals torch tensors into it.  ``workloads`` holds the synthetic input
recipes.  Importing the package does not load the CUDA library; the first call does,
and raises if it is missing.
"""

__all__ = ["binding", "workloads"]
