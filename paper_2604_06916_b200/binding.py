"""ctypes binding of the C-ABI CUDA library (``include/sol_nvfp4.h``).

Argument marshalling only: torch supplies device memory and the current stream, every
compute step runs in the library's kernels.  There is no fallback: if the library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import functools
import os
import types

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("SOL_NVFP4_LIB", os.path.join(_HERE, "libsol_nvfp4.so"))

SF_ROW_MAJOR = 0
SF_SWIZZLED_128x4 = 1

EXPORTS = [
    "sol_status_string", "sol_nvfp4_data_bytes", "sol_nvfp4_scale_bytes",
    "sol_nvfp4_linear_workspace_bytes", "sol_amax_bf16", "nvfp4_quantize", "nvfp4_quantize_weight",
    "nvfp4_linear", "bf16_linear", "nvfp4_quantize_linear", "sol_last_device_status",
    "sol_nvfp4_static_scratch_bytes", "nvfp4_quantize_linear_static", "nvfp4_quantize_linear_host",
    "nvfp4_requantize_lora", "nvfp4_requantize_lora_batch", "nvfp4_linear_quantized_out",
    "solrl_select_contrastive", "solrl_rank_consistency", "sol_mxfp4_scale_bytes", "mxfp4_quantize",
    "mxfp4_linear", "nvfp4_linear_split_out", "nvfp4_quantize_into",
    "nvfp4_quantize_linear_delayed", "sol_roll_tensor_scale", "nvfp4_layernorm_quantize", "sol_attention_bf16", "sol_attention_bf16_joint",
    "sol_attention_nvfp4_out", "mxfp4_linear_quantized_out", "sol_set_wait_limit_cycles", "sol_test_hold_loads",
    "mxfp4_linear_split_out", "mxfp4_quantize_into",
]

_lib = None


class SolError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


def lib() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2604_06916_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i64, sz, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t, ctypes.c_int
    L.sol_status_string.restype, L.sol_status_string.argtypes = ctypes.c_char_p, [i32]
    L.sol_nvfp4_data_bytes.restype, L.sol_nvfp4_data_bytes.argtypes = sz, [i64, i64]
    L.sol_nvfp4_scale_bytes.restype, L.sol_nvfp4_scale_bytes.argtypes = sz, [i64, i64, i32]
    L.sol_nvfp4_linear_workspace_bytes.restype = sz
    L.sol_nvfp4_linear_workspace_bytes.argtypes = [i64, i64, i64]
    L.sol_amax_bf16.restype, L.sol_amax_bf16.argtypes = i32, [vp, i64, i64, i64, vp, vp]
    L.nvfp4_quantize.restype, L.nvfp4_quantize.argtypes = i32, [vp, i64, i64, i64, vp, vp, vp, i32, vp]
    L.nvfp4_quantize_weight.restype = i32
    L.nvfp4_quantize_weight.argtypes = [vp, i64, i64, i64, vp, vp, vp, i32, vp]
    L.nvfp4_linear.restype = i32
    L.nvfp4_linear.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, vp]
    L.bf16_linear.restype = i32
    L.bf16_linear.argtypes = [vp, vp, vp, vp, i64, i64, i64, i64, i64, i64, vp]
    L.nvfp4_quantize_linear.restype = i32
    L.nvfp4_quantize_linear.argtypes = [vp, i64, vp, vp, vp, vp, vp, i64, i64, i64, i64, vp, sz, vp]
    L.sol_nvfp4_static_scratch_bytes.restype, L.sol_nvfp4_static_scratch_bytes.argtypes = sz, []
    L.nvfp4_quantize_linear_static.restype = i32
    L.nvfp4_quantize_linear_static.argtypes = [vp, i64, vp, vp, vp, vp, vp, i64, i64, i64, i64, vp]
    L.nvfp4_quantize_linear_host.restype = i32
    L.nvfp4_quantize_linear_host.argtypes = [vp, i64, vp, vp, vp, vp, vp, i64, i64, i64, i64, vp, vp, vp, sz, vp]
    L.nvfp4_requantize_lora.restype = i32
    L.nvfp4_requantize_lora.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, i64, ctypes.c_float, vp, vp, vp, vp,
                                        i32, vp]
    L.nvfp4_requantize_lora_batch.restype = i32
    L.nvfp4_requantize_lora_batch.argtypes = [i64, vp, vp, vp, vp, vp, vp, i64, i64, i64, ctypes.c_float, vp, i64,
                                              i32, vp]
    L.nvfp4_linear_quantized_out.restype = i32
    L.nvfp4_linear_quantized_out.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, i64, i64, i64, vp]
    L.solrl_select_contrastive.restype = i32
    L.solrl_select_contrastive.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp, vp]
    L.solrl_rank_consistency.restype = i32
    L.solrl_rank_consistency.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp]
    L.sol_mxfp4_scale_bytes.restype, L.sol_mxfp4_scale_bytes.argtypes = sz, [i64, i64, i32]
    L.mxfp4_quantize.restype, L.mxfp4_quantize.argtypes = i32, [vp, i64, i64, i64, vp, vp, i32, vp]
    L.mxfp4_linear.restype, L.mxfp4_linear.argtypes = i32, [vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, vp]
    L.nvfp4_linear_split_out.restype = i32
    L.nvfp4_linear_split_out.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, i32, vp, vp, vp, i64, i64, vp, i64,
                                         i64, i64, vp]
    L.nvfp4_quantize_into.restype = i32
    L.nvfp4_quantize_into.argtypes = [vp, i64, i64, i64, vp, vp, vp, i64, i64, vp]
    L.nvfp4_quantize_linear_delayed.restype = i32
    L.nvfp4_quantize_linear_delayed.argtypes = [vp, i64, vp, vp, vp, vp, vp, i64, i64, i64, i64, vp, vp, sz, vp]
    L.sol_roll_tensor_scale.restype, L.sol_roll_tensor_scale.argtypes = i32, [vp, vp]
    L.sol_attention_bf16_joint.restype = i32
    L.sol_attention_bf16_joint.argtypes = [ctypes.POINTER(AttentionStream), ctypes.POINTER(AttentionStream), i64, i64, i64, vp]
    L.mxfp4_linear_quantized_out.restype = i32
    L.mxfp4_linear_quantized_out.argtypes = [vp, vp, vp, vp, vp, i32, vp, vp, vp, i64, i64, i64, vp]
    L.sol_attention_nvfp4_out.restype = i32
    L.sol_attention_nvfp4_out.argtypes = [vp, vp, vp, i64, i64, i64, i64, i64, i64, i64, i64, vp, vp, vp, i64, i64, vp, vp]
    L.sol_attention_bf16.restype = i32
    L.sol_attention_bf16.argtypes = [vp, vp, vp, vp, i64, i64, i64, i64, i64, i64, i64, i64, i64, vp]
    L.nvfp4_layernorm_quantize.restype = i32
    L.nvfp4_layernorm_quantize.argtypes = [vp, i64, i64, i64, vp, vp, i64, ctypes.c_float, vp, vp, vp, vp, vp]
    L.mxfp4_linear_split_out.restype = i32
    L.mxfp4_linear_split_out.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i32, vp, vp, i64, i64, vp, i64, i64, i64, vp]
    L.mxfp4_quantize_into.restype = i32
    L.mxfp4_quantize_into.argtypes = [vp, i64, i64, i64, vp, vp, i64, i64, vp]
    L.sol_set_wait_limit_cycles.restype, L.sol_set_wait_limit_cycles.argtypes = i32, [i64]
    L.sol_test_hold_loads.restype, L.sol_test_hold_loads.argtypes = i32, [i32]
    L.sol_last_device_status.restype = i32
    L.sol_last_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    _lib = L
    return L


def status_string(code: int) -> str:
    return lib().sol_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != 0:
        raise SolError(code, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


# Guard bands (debugging aid, off unless SOL_NVFP4_GUARD=1): every output this module allocates sits between
# two 4 KB bands of a fixed byte, and after each call the device is synchronised and the bands are checked, so
# a kernel that writes outside its output is caught by the call that did it.  Callers' own `out=` buffers
# are theirs to guard.
GUARD_BYTES = 4096
GUARD_BYTE = 0xA5
_guard_pending: list = []


def guard_mode() -> bool:
    return os.environ.get("SOL_NVFP4_GUARD", "0") not in ("", "0")


def _empty(shape, dtype, device) -> torch.Tensor:
    """torch.empty, or (guard mode) a view between two guard bands of one larger allocation."""
    if not guard_mode():
        return torch.empty(shape, dtype=dtype, device=device)
    shape = (shape,) if isinstance(shape, int) else tuple(shape)
    n = 1
    for d in shape:
        n *= int(d)
    nbytes = n * torch.empty((), dtype=dtype).element_size()
    padded = (nbytes + 255) // 256 * 256          # the back band starts on a 256-byte boundary
    raw = torch.empty(2 * GUARD_BYTES + padded, dtype=torch.uint8, device=device)
    raw[:GUARD_BYTES].fill_(GUARD_BYTE)
    raw[GUARD_BYTES + nbytes:].fill_(GUARD_BYTE)
    _guard_pending.append((raw, nbytes))
    return raw[GUARD_BYTES:GUARD_BYTES + nbytes].view(dtype).view(shape)


def check_guards(where: str = "") -> None:
    """Verify and forget the guard bands of the outputs allocated since the last check."""
    pending, bad = list(_guard_pending), []
    _guard_pending.clear()
    if not pending:
        return
    if pending[0][0].is_cuda:
        torch.cuda.synchronize()
    for raw, nbytes in pending:
        front = bool((raw[:GUARD_BYTES] == GUARD_BYTE).all())
        back = bool((raw[GUARD_BYTES + nbytes:] == GUARD_BYTE).all())
        if not (front and back):
            bad.append(f"{nbytes}-byte output: {'front' if not front else 'back'} band overwritten")
    if bad:
        raise AssertionError(f"{where}: write outside an output buffer ({'; '.join(bad)})")


def _guarded(fn):
    @functools.wraps(fn)
    def call(*args, **kwargs):
        if not guard_mode():
            return fn(*args, **kwargs)
        try:
            return fn(*args, **kwargs)
        finally:
            check_guards(fn.__name__)
    return call


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def data_bytes(rows: int, K: int) -> int:
    return lib().sol_nvfp4_data_bytes(rows, K)


def scale_bytes(rows: int, K: int, layout: int = SF_SWIZZLED_128x4) -> int:
    return lib().sol_nvfp4_scale_bytes(rows, K, layout)


def linear_workspace_bytes(M: int, N: int, K: int) -> int:
    return lib().sol_nvfp4_linear_workspace_bytes(M, N, K)


def _need_2d_bf16(x: torch.Tensor, name: str):
    if x.dtype != torch.bfloat16 or x.dim() != 2 or x.stride(1) != 1 or not x.is_cuda:
        raise TypeError(f"{name}: expected a 2-D CUDA bf16 tensor with contiguous rows")


def sol_amax_bf16(x: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """Per-tensor scale T = max|x| / 2688 (1 for zeros) as a 1-element float32 device tensor."""
    _need_2d_bf16(x, "x")
    if out is None:
        out = _empty(1, torch.float32, x.device)
    _check(lib().sol_amax_bf16(_ptr(x), x.shape[0], x.shape[1], x.stride(0), _ptr(out), _stream()), "sol_amax_bf16")
    return out


def _alloc_q(rows: int, K: int, layout: int, device):
    nq, ns = data_bytes(rows, K), scale_bytes(rows, K, layout)
    if nq == 0 or ns == 0:
        raise SolError(2, "shape check")
    q = _empty((rows, K // 2), torch.uint8, device)
    sf = _empty(ns, torch.uint8, device)
    return q, sf


def nvfp4_quantize(x: torch.Tensor, tensor_scale: torch.Tensor, layout: int = SF_SWIZZLED_128x4,
                   out: tuple[torch.Tensor, torch.Tensor] | None = None):
    """BF16 [M, K] -> (packed nibbles uint8 [M, K/2], E4M3 scales uint8 flat buffer)."""
    _need_2d_bf16(x, "x")
    M, K = x.shape
    q, sf = out if out is not None else _alloc_q(M, K, layout, x.device)
    _check(lib().nvfp4_quantize(_ptr(x), M, K, x.stride(0), _ptr(tensor_scale), _ptr(q), _ptr(sf), layout,
                                _stream()), "nvfp4_quantize")
    return q, sf


def nvfp4_quantize_weight(w: torch.Tensor, layout: int = SF_SWIZZLED_128x4):
    """BF16 [N, K] -> (packed nibbles, scales, per-tensor scale T_w)."""
    _need_2d_bf16(w, "w")
    N, K = w.shape
    q, sf = _alloc_q(N, K, layout, w.device)
    ts = _empty(1, torch.float32, w.device)
    _check(lib().nvfp4_quantize_weight(_ptr(w), N, K, w.stride(0), _ptr(q), _ptr(sf), _ptr(ts), layout, _stream()),
           "nvfp4_quantize_weight")
    return q, sf, ts


def nvfp4_requantize_lora(w: torch.Tensor, lora_a: torch.Tensor, lora_b: torch.Tensor, scaling: float,
                          layout: int = SF_SWIZZLED_128x4, merged: torch.Tensor | None = None, out=None):
    """Merge adapters (W + scaling * B A, BF16) and quantize: (merged W', nibbles, scales, T).

    ``out`` = (q, sf, ts) supplies the output buffers; ts holds two floats (T and the entry
    point's scratch word), the returned T is a view of its first element.
    """
    _need_2d_bf16(w, "w")
    _need_2d_bf16(lora_a, "lora_a")
    _need_2d_bf16(lora_b, "lora_b")
    N, K = w.shape
    r = lora_a.shape[0]
    if lora_a.shape[1] != K or tuple(lora_b.shape) != (N, r):
        raise ValueError("shapes: w [N, K], lora_a [r, K], lora_b [N, r]")
    if merged is None:
        merged = _empty((N, K), torch.bfloat16, w.device)
    if out is None:
        q, sf = _alloc_q(N, K, layout, w.device)
        ts2 = _empty(2, torch.float32, w.device)
    else:
        q, sf, ts2 = out
        if ts2.numel() < 2:
            raise ValueError("ts must hold two floats")
    _check(lib().nvfp4_requantize_lora(_ptr(w), w.stride(0), _ptr(lora_a), lora_a.stride(0), _ptr(lora_b),
                                       lora_b.stride(0), N, K, r, float(scaling), _ptr(merged), _ptr(q),
                                       _ptr(sf), _ptr(ts2), layout, _stream()), "nvfp4_requantize_lora")
    return merged, q, sf, ts2[:1]


class LoraRefreshPlan:
    """Pointer lists for nvfp4_requantize_lora_batch, built once for a set of same-shaped matrices.

    ``items`` = [(w, lora_a, lora_b), ...]; the outputs (q, sf, ts) are allocated here and kept in
    ``outputs``; ``run()`` re-quantizes all of them with one call into the library, ``group``
    matrices per launch (the merged-weight scratch holds that many).
    """

    def __init__(self, items, scaling: float, layout: int = SF_SWIZZLED_128x4, group: int = 8):
        if not items:
            raise ValueError("no matrices")
        N, K = items[0][0].shape
        r = items[0][1].shape[0]
        for w, a, b in items:
            for t, name in ((w, "w"), (a, "lora_a"), (b, "lora_b")):
                _need_2d_bf16(t, name)
                if not t.is_contiguous():
                    raise ValueError(f"{name} must be dense")
            if tuple(w.shape) != (N, K) or tuple(a.shape) != (r, K) or tuple(b.shape) != (N, r):
                raise ValueError("all matrices of a plan share one shape")
        dev = items[0][0].device
        self.items = list(items)
        self.N, self.K, self.r, self.scaling, self.layout = N, K, r, float(scaling), layout
        self.group = max(1, min(group, len(items)))
        self.merged = _empty((self.group, N, K), torch.bfloat16, dev)
        self.outputs = []
        for _ in items:
            q, sf = _alloc_q(N, K, layout, dev)
            self.outputs.append((q, sf, _empty(2, torch.float32, dev)))
        n = len(items)
        arr = ctypes.c_void_p * n
        self._lists = [arr(*[t[i].data_ptr() for t in items]) for i in range(3)] + \
                      [arr(*[o[i].data_ptr() for o in self.outputs]) for i in range(3)]

    def run(self):
        _check(lib().nvfp4_requantize_lora_batch(len(self.items), *self._lists, self.N, self.K, self.r,
                                                 self.scaling, _ptr(self.merged), self.group, self.layout, _stream()),
               "nvfp4_requantize_lora_batch")
        return self.outputs


def nvfp4_linear(xq, xsf, x_tscale, wq, wsf, w_tscale, bias=None, out: torch.Tensor | None = None):
    """Y = dequant(X) . dequant(W)^T + bias in BF16 from quantized operands (swizzled scales)."""
    M, K = xq.shape[0], xq.shape[1] * 2
    N = wq.shape[0]
    if out is None:
        out = _empty((M, N), torch.bfloat16, xq.device)
    _check(lib().nvfp4_linear(_ptr(xq), _ptr(xsf), _ptr(x_tscale), _ptr(wq), _ptr(wsf), _ptr(w_tscale), _ptr(bias),
                              _ptr(out), M, N, K, out.stride(0), _stream()), "nvfp4_linear")
    return out


ACT_NONE, ACT_GELU_TANH = 0, 1


def nvfp4_linear_split_out(xq, xsf, x_tscale, wq, wsf, w_tscale, bias, n_split: int, activation: int, out_tscale,
                           dest, dest_col0: int, y_out: torch.Tensor | None = None,
                           amax_out: torch.Tensor | None = None):
    """Columns below n_split -> BF16 `y_out`; the rest -> activation -> quantized into dest = (q [M, dest_K/2], sf)."""
    M, K = xq.shape[0], xq.shape[1] * 2
    N = wq.shape[0]
    hq, hsf = dest
    dest_K = hq.shape[1] * 2
    if y_out is None:
        y_out = _empty((M, n_split), torch.bfloat16, xq.device)
    _check(lib().nvfp4_linear_split_out(_ptr(xq), _ptr(xsf), _ptr(x_tscale), _ptr(wq), _ptr(wsf), _ptr(w_tscale),
                                        _ptr(bias), _ptr(y_out), y_out.stride(0), n_split, activation, _ptr(out_tscale),
                                        _ptr(hq), _ptr(hsf), dest_K, dest_col0, _ptr(amax_out), M, N, K, _stream()),
           "nvfp4_linear_split_out")
    return y_out


def nvfp4_quantize_into(x: torch.Tensor, tensor_scale: torch.Tensor, dest, dest_col0: int):
    """Quantize BF16 x [M, K] into columns [dest_col0, dest_col0 + K) of dest = (q [M, dest_K/2], sf)."""
    _need_2d_bf16(x, "x")
    M, K = x.shape
    hq, hsf = dest
    _check(lib().nvfp4_quantize_into(_ptr(x), M, K, x.stride(0), _ptr(tensor_scale), _ptr(hq), _ptr(hsf),
                                     hq.shape[1] * 2, dest_col0, _stream()), "nvfp4_quantize_into")


def nvfp4_quantize_linear_delayed(x, wq, wsf, w_tscale, bias, scale_state: torch.Tensor,
                                  workspace: torch.Tensor | None = None, out: torch.Tensor | None = None):
    """Fused quantize + NVFP4 linear with T = scale_state[0]; max|x| is accumulated into scale_state[1]."""
    _need_2d_bf16(x, "x")
    M, K = x.shape
    N = wq.shape[0]
    if workspace is None:
        workspace = _empty(linear_workspace_bytes(M, N, K), torch.uint8, x.device)
    if out is None:
        out = _empty((M, N), torch.bfloat16, x.device)
    _check(lib().nvfp4_quantize_linear_delayed(_ptr(x), x.stride(0), _ptr(wq), _ptr(wsf), _ptr(w_tscale), _ptr(bias),
                                               _ptr(out), M, N, K, out.stride(0), _ptr(scale_state), _ptr(workspace),
                                               workspace.numel(), _stream()), "nvfp4_quantize_linear_delayed")
    return out


def sol_roll_tensor_scale(scale_state: torch.Tensor):
    _check(lib().sol_roll_tensor_scale(_ptr(scale_state), _stream()), "sol_roll_tensor_scale")


def nvfp4_layernorm_quantize(x, scale, shift, rows_per_sample: int, tensor_scale, eps: float = 1e-6,
                             amax_out: torch.Tensor | None = None, out=None):
    """LN(x) * (1 + scale[sample]) + shift[sample], quantized for the next linear: (nibbles, swizzled scales)."""
    _need_2d_bf16(x, "x")
    _need_2d_bf16(scale, "scale")
    _need_2d_bf16(shift, "shift")
    M, K = x.shape
    if out is None:
        out = _alloc_q(M, K, SF_SWIZZLED_128x4, x.device)
    q, sf = out
    _check(lib().nvfp4_layernorm_quantize(_ptr(x), M, K, x.stride(0), _ptr(scale), _ptr(shift), rows_per_sample,
                                          float(eps), _ptr(tensor_scale), _ptr(q), _ptr(sf), _ptr(amax_out), _stream()),
           "nvfp4_layernorm_quantize")
    return q, sf


class AttentionStream(ctypes.Structure):
    """sol_attention_stream_t of the C header."""
    _fields_ = [("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("out", ctypes.c_void_p),
                ("seq", ctypes.c_int64), ("ld_q", ctypes.c_int64), ("ld_k", ctypes.c_int64), ("ld_v", ctypes.c_int64),
                ("ld_out", ctypes.c_int64)]


def _token_pitch(t: torch.Tensor) -> int:
    """Elements between consecutive tokens of a [B, S, H, D] view (a dimension of extent 1 has no meaningful stride)."""
    if t.shape[1] > 1:
        return t.stride(1)
    return t.stride(0) if t.shape[0] > 1 else t.shape[2] * t.shape[3]


def _check_attention_view(name: str, t: torch.Tensor):
    if t.dtype != torch.bfloat16 or t.dim() != 4 or t.shape[3] not in (64, 128):
        raise ValueError(f"{name} must be a [B, S, H, D] BF16 tensor with D = 64 or 128")
    if t.stride(3) != 1 or (t.shape[2] > 1 and t.stride(2) != t.shape[3]) or \
            (t.shape[0] > 1 and t.shape[1] > 1 and t.stride(0) != t.shape[1] * t.stride(1)):
        raise ValueError(f"{name}: heads and head dimension must be contiguous, batches stacked densely")


def sol_attention_bf16_joint(first, second, out=None):
    """Joint attention of two token streams: first = (q, k, v) of the stream whose tokens come first.

    Every tensor is a [B, S_stream, H, D] view as in sol_attention_bf16; S of the first stream is a
    multiple of 256.  Returns (out_first, out_second), each [B, S_stream, H, D].
    """
    streams = []
    outs = list(out) if out is not None else [None, None]
    for i, (q, k, v) in enumerate((first, second)):
        for name, t in (("q", q), ("k", k), ("v", v)):
            _check_attention_view(name, t)
        if q.shape != k.shape or q.shape != v.shape:
            raise ValueError("q, k and v of a stream must have one shape")
        if outs[i] is None:
            outs[i] = _empty(tuple(q.shape), torch.bfloat16, q.device)
        _check_attention_view("out", outs[i])
        streams.append(AttentionStream(_ptr(q), _ptr(k), _ptr(v), _ptr(outs[i]), q.shape[1], _token_pitch(q),
                                       _token_pitch(k), _token_pitch(v), _token_pitch(outs[i])))
    B_, _, H, D = first[0].shape
    if second[0].shape[0] != B_ or second[0].shape[2] != H or second[0].shape[3] != D:
        raise ValueError("both streams must share batch, heads and head dimension")
    _check(lib().sol_attention_bf16_joint(ctypes.byref(streams[0]), ctypes.byref(streams[1]), B_, H, D, _stream()),
           "sol_attention_bf16_joint")
    return outs[0], outs[1]


def sol_attention_bf16(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor | None = None):
    """softmax(q k^T / sqrt(D)) v per batch element and head, D = 64 or 128.

    q [B, Sq, H, D], k and v [B, Skv, H, D], BF16; the last two dimensions contiguous, the batch
    dimension densely on top of the token dimension (stride(0) == S * stride(1)) -- views into a fused
    projection output qualify.  Returns [B, Sq, H, D].
    """
    for name, t in (("q", q), ("k", k), ("v", v)):
        _check_attention_view(name, t)
    B, Sq, H, D = q.shape
    if k.shape != v.shape or k.shape[0] != B or k.shape[2] != H or k.shape[3] != D:
        raise ValueError("k and v must share [B, Skv, H, D] with q's batch, heads and head dimension")
    if out is None:
        out = _empty((B, Sq, H, D), torch.bfloat16, q.device)
    _check_attention_view("out", out)
    _check(lib().sol_attention_bf16(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, Sq, k.shape[1], H, D, _token_pitch(q),
                                    _token_pitch(k), _token_pitch(v), _token_pitch(out), _stream()), "sol_attention_bf16")
    return out


def sol_attention_nvfp4_out(q, k, v, out_tscale: torch.Tensor, dest, dest_col0: int = 0,
                            amax_out: torch.Tensor | None = None):
    """Attention whose output is quantized into columns [dest_col0, dest_col0 + H * D) of `dest`.

    dest = (nibbles [B * Sq, dest_K / 2] uint8, swizzled scales of a [B * Sq, dest_K] tensor); returns dest.
    """
    for name, t in (("q", q), ("k", k), ("v", v)):
        _check_attention_view(name, t)
    B, Sq, H, D = q.shape
    if k.shape != v.shape or k.shape[0] != B or k.shape[2] != H or k.shape[3] != D:
        raise ValueError("k and v must share [B, Skv, H, D] with q's batch, heads and head dimension")
    dq, dsf = dest
    if dq.dtype != torch.uint8 or dq.dim() != 2 or dq.shape[0] != B * Sq or not dq.is_contiguous():
        raise ValueError("dest nibbles must be a contiguous [B * Sq, dest_K / 2] uint8 tensor")
    _check(lib().sol_attention_nvfp4_out(_ptr(q), _ptr(k), _ptr(v), B, Sq, k.shape[1], H, D, _token_pitch(q), _token_pitch(k),
                                         _token_pitch(v), _ptr(out_tscale), _ptr(dq), _ptr(dsf), dq.shape[1] * 2, dest_col0,
                                         _ptr(amax_out), _stream()), "sol_attention_nvfp4_out")
    return dest


def mxfp4_scale_bytes(rows: int, K: int, layout: int = SF_SWIZZLED_128x4) -> int:
    return int(lib().sol_mxfp4_scale_bytes(rows, K, layout))


def mxfp4_quantize(x: torch.Tensor, layout: int = SF_SWIZZLED_128x4, out=None):
    """BF16 [rows, K] -> (packed nibbles [rows, K/2], E8M0 scales in the given layout)."""
    _need_2d_bf16(x, "x")
    rows, K = x.shape
    if out is None:
        nbytes = mxfp4_scale_bytes(rows, K, layout)
        if nbytes == 0:
            raise ValueError("bad shape for mxfp4_quantize")
        out = (_empty((rows, K // 2), torch.uint8, x.device),
               _empty(nbytes, torch.uint8, x.device))
    q, sf = out
    _check(lib().mxfp4_quantize(_ptr(x), rows, K, x.stride(0), _ptr(q), _ptr(sf), layout, _stream()), "mxfp4_quantize")
    return q, sf


def mxfp4_linear(xq, xsf, wq, wsf, bias=None, out: torch.Tensor | None = None):
    """Y = dequant(X) . dequant(W)^T + bias in BF16 from MXFP4 operands (chunked scales)."""
    M, K = xq.shape[0], xq.shape[1] * 2
    N = wq.shape[0]
    if out is None:
        out = _empty((M, N), torch.bfloat16, xq.device)
    _check(lib().mxfp4_linear(_ptr(xq), _ptr(xsf), _ptr(wq), _ptr(wsf), _ptr(bias), _ptr(out), M, N, K, out.stride(0),
                              _stream()), "mxfp4_linear")
    return out


def mxfp4_linear_split_out(xq, xsf, wq, wsf, bias, n_split: int, activation: int, dest, dest_col0: int,
                           y_out: torch.Tensor | None = None, amax_out: torch.Tensor | None = None):
    """Columns below n_split -> BF16 `y_out`; the rest -> activation -> MXFP4 into dest = (q [M, dest_K/2], sf)."""
    M, K = xq.shape[0], xq.shape[1] * 2
    N = wq.shape[0]
    hq, hsf = dest
    if y_out is None:
        y_out = _empty((M, n_split), torch.bfloat16, xq.device)
    _check(lib().mxfp4_linear_split_out(_ptr(xq), _ptr(xsf), _ptr(wq), _ptr(wsf), _ptr(bias), _ptr(y_out), y_out.stride(0),
                                        n_split, activation, _ptr(hq), _ptr(hsf), hq.shape[1] * 2, dest_col0,
                                        _ptr(amax_out), M, N, K, _stream()), "mxfp4_linear_split_out")
    return y_out


def mxfp4_quantize_into(x: torch.Tensor, dest, dest_col0: int):
    """Quantize BF16 x [M, K] into columns [dest_col0, dest_col0 + K) of the MXFP4 tensor dest = (q, sf)."""
    _need_2d_bf16(x, "x")
    M, K = x.shape
    hq, hsf = dest
    _check(lib().mxfp4_quantize_into(_ptr(x), M, K, x.stride(0), _ptr(hq), _ptr(hsf), hq.shape[1] * 2, dest_col0,
                                     _stream()), "mxfp4_quantize_into")


def solrl_select_contrastive(rewards: torch.Tensor, K: int, seeds: torch.Tensor | None = None,
                             with_advantages: bool = True):
    """[P, N] FP32 rewards -> (indices [P, K] int32, selected seeds or None, advantages [P, N] or None)."""
    if rewards.dtype != torch.float32 or rewards.dim() != 2 or not rewards.is_contiguous():
        raise ValueError("rewards must be a dense 2-D float32 tensor")
    P, N = rewards.shape
    idx = _empty((P, K), torch.int32, rewards.device)
    sel = None
    if seeds is not None:
        if seeds.dtype != torch.int64 or tuple(seeds.shape) != (P, N) or not seeds.is_contiguous():
            raise ValueError("seeds must be a dense [P, N] int64 tensor")
        sel = _empty((P, K), torch.int64, rewards.device)
    adv = torch.empty_like(rewards) if with_advantages else None
    _check(lib().solrl_select_contrastive(_ptr(rewards), _ptr(seeds), P, N, K, _ptr(idx), _ptr(sel), _ptr(adv),
                                          _stream()), "solrl_select_contrastive")
    return idx, sel, adv


def solrl_rank_consistency(ref: torch.Tensor, proxy: torch.Tensor, k: int):
    """Per prompt: exact counts [P, 4] int64 and (tau, rho, top-k match, bottom-k match) [P, 4] FP32."""
    for t in (ref, proxy):
        if t.dtype != torch.float32 or t.dim() != 2 or not t.is_contiguous():
            raise ValueError("rewards must be dense 2-D float32 tensors")
    if ref.shape != proxy.shape:
        raise ValueError("shapes differ")
    P, N = ref.shape
    counts = _empty((P, 4), torch.int64, ref.device)
    metrics = _empty((P, 4), torch.float32, ref.device)
    _check(lib().solrl_rank_consistency(_ptr(ref), _ptr(proxy), P, N, k, _ptr(counts), _ptr(metrics), _stream()),
           "solrl_rank_consistency")
    return counts, metrics


def nvfp4_linear_quantized_out(xq, xsf, x_tscale, wq, wsf, w_tscale, bias, activation: int, out_tscale,
                               amax_out: torch.Tensor | None = None, out=None):
    """NVFP4 linear whose output leaves as (nibbles [M, N/2], swizzled scales) for the next linear."""
    M, K = xq.shape[0], xq.shape[1] * 2
    N = wq.shape[0]
    if out is None:
        out = _alloc_q(M, N, SF_SWIZZLED_128x4, xq.device)
    hq, hsf = out
    _check(lib().nvfp4_linear_quantized_out(_ptr(xq), _ptr(xsf), _ptr(x_tscale), _ptr(wq), _ptr(wsf), _ptr(w_tscale),
                                            _ptr(bias), activation, _ptr(out_tscale), _ptr(hq), _ptr(hsf),
                                            _ptr(amax_out), M, N, K, _stream()), "nvfp4_linear_quantized_out")
    return hq, hsf


def mxfp4_linear_quantized_out(xq, xsf, wq, wsf, bias, activation: int, amax_out: torch.Tensor | None = None, out=None):
    """MXFP4 linear whose output leaves as (nibbles [M, N/2], swizzled E8M0 scales) for the next MXFP4 linear."""
    M, K = xq.shape[0], xq.shape[1] * 2
    N = wq.shape[0]
    if out is None:
        out = (_empty((M, N // 2), torch.uint8, xq.device),
               _empty(mxfp4_scale_bytes(M, N), torch.uint8, xq.device))
    hq, hsf = out
    _check(lib().mxfp4_linear_quantized_out(_ptr(xq), _ptr(xsf), _ptr(wq), _ptr(wsf), _ptr(bias), activation, _ptr(hq),
                                            _ptr(hsf), _ptr(amax_out), M, N, K, _stream()), "mxfp4_linear_quantized_out")
    return hq, hsf


def bf16_linear(x, w, bias=None, out: torch.Tensor | None = None):
    """Y = X . W^T + bias, BF16 in / BF16 out, FP32 accumulation."""
    _need_2d_bf16(x, "x")
    _need_2d_bf16(w, "w")
    M, K = x.shape
    N = w.shape[0]
    if out is None:
        out = _empty((M, N), torch.bfloat16, x.device)
    _check(lib().bf16_linear(_ptr(x), _ptr(w), _ptr(bias), _ptr(out), M, N, K, x.stride(0), w.stride(0),
                             out.stride(0), _stream()), "bf16_linear")
    return out


def nvfp4_quantize_linear(x, wq, wsf, w_tscale, bias=None, workspace: torch.Tensor | None = None,
                          out: torch.Tensor | None = None):
    """Dynamic per-tensor scale + quantize X + NVFP4 GEMM against pre-quantized W, one call."""
    _need_2d_bf16(x, "x")
    M, K = x.shape
    N = wq.shape[0]
    if workspace is None:
        workspace = _empty(linear_workspace_bytes(M, N, K), torch.uint8, x.device)
    if out is None:
        out = _empty((M, N), torch.bfloat16, x.device)
    _check(lib().nvfp4_quantize_linear(_ptr(x), x.stride(0), _ptr(wq), _ptr(wsf), _ptr(w_tscale), _ptr(bias),
                                       _ptr(out), M, N, K, out.stride(0), _ptr(workspace), workspace.numel(),
                                       _stream()), "nvfp4_quantize_linear")
    return out


def nvfp4_quantize_linear_host(x_host, wq, wsf, w_tscale, bias, y_host, x_dev, y_dev, workspace):
    """End-to-end form: host X (ideally pinned) -> device, fused quantize + NVFP4 linear, Y -> host."""
    M, K = x_host.shape
    N = wq.shape[0]
    _check(lib().nvfp4_quantize_linear_host(_ptr(x_host), x_host.stride(0), _ptr(wq), _ptr(wsf), _ptr(w_tscale),
                                            _ptr(bias), _ptr(y_host), M, N, K, y_host.stride(0), _ptr(x_dev),
                                            _ptr(y_dev), _ptr(workspace), workspace.numel(), _stream()),
           "nvfp4_quantize_linear_host")
    return y_host


def static_scratch_bytes() -> int:
    return lib().sol_nvfp4_static_scratch_bytes()


def nvfp4_quantize_linear_static(x, wq, wsf, w_tscale, bias=None, out: torch.Tensor | None = None):
    """nvfp4_quantize_linear for callers that may not allocate: the scratch is a fixed array inside
    the library (64 MiB, shared by every call on the device; overlapping calls race).  Only the output
    tensor is created here when `out` is not given -- pass `out` to allocate nothing at all."""
    _need_2d_bf16(x, "x")
    M, K = x.shape
    N = wq.shape[0]
    if out is None:
        out = _empty((M, N), torch.bfloat16, x.device)
    _check(lib().nvfp4_quantize_linear_static(_ptr(x), x.stride(0), _ptr(wq), _ptr(wsf), _ptr(w_tscale), _ptr(bias),
                                              _ptr(out), M, N, K, out.stride(0), _stream()),
           "nvfp4_quantize_linear_static")
    return out


def sol_last_device_status() -> int:
    """Synchronises the current stream; raises SolError if a bounded device wait ran out."""
    detail = ctypes.c_uint32(0)
    code = lib().sol_last_device_status(_stream(), ctypes.byref(detail))
    if code != 0:
        err = SolError(code, f"device status word 0x{detail.value:x}")
        err.detail = detail.value
        raise err
    return 0


def sol_set_wait_limit_cycles(cycles: int) -> None:
    """Limit of every bounded device-side wait on the current device, in SM cycles (<= 0: default)."""
    _check(lib().sol_set_wait_limit_cycles(int(cycles)), "sol_set_wait_limit_cycles")


def sol_test_hold_loads(on: bool) -> None:
    """Test hook: while on, the pair GEMM kernels issue no loads and their waits run into the limit."""
    _check(lib().sol_test_hold_loads(1 if on else 0), "sol_test_hold_loads")


# every public entry checks the guard bands of what it allocated (a no-op outside guard mode)
for _name, _fn in list(globals().items()):
    if (isinstance(_fn, types.FunctionType) and _fn.__module__ == __name__ and not _name.startswith("_")
            and _name not in ("lib", "guard_mode", "check_guards", "status_string")):
        globals()[_name] = _guarded(_fn)
del _name, _fn
