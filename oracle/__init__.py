"""CPU oracle for the NVFP4 linear path -- TEST INFRASTRUCTURE, not a product path.

Thin ctypes/numpy access to ``nvfp4_oracle.c`` (plain C, FP32 steps for the
quantizer, FP64 for the matmuls).  Only the tests, the smoke check and the CPU
baseline leg of the benchmark may import this package; the CUDA library never
does, and nothing here imports the CUDA library.

BF16 tensors are passed as ``numpy.uint16`` bit patterns, packed FP4 data and
E4M3 scales as ``numpy.uint8``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nvfp4_oracle.c")
_LIB = os.path.join(_HERE, "libnvfp4_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (strict IEEE: no contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    L = ctypes.CDLL(_LIB)
    u8p, u16p = ctypes.POINTER(ctypes.c_uint8), ctypes.POINTER(ctypes.c_uint16)
    f64p, i64p = ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64)
    i64, f32 = ctypes.c_int64, ctypes.c_float
    L.oracle_bf16_to_f32.restype, L.oracle_bf16_to_f32.argtypes = f32, [ctypes.c_uint16]
    L.oracle_f64_to_bf16.restype, L.oracle_f64_to_bf16.argtypes = ctypes.c_uint16, [ctypes.c_double]
    L.oracle_e2m1_decode.restype, L.oracle_e2m1_decode.argtypes = ctypes.c_double, [ctypes.c_uint8]
    L.oracle_e2m1_encode.restype, L.oracle_e2m1_encode.argtypes = ctypes.c_uint8, [f32]
    L.oracle_e4m3_decode.restype, L.oracle_e4m3_decode.argtypes = ctypes.c_double, [ctypes.c_uint8]
    L.oracle_e4m3_encode.restype, L.oracle_e4m3_encode.argtypes = ctypes.c_uint8, [f32]
    L.oracle_tensor_scale.restype, L.oracle_tensor_scale.argtypes = f32, [u16p, i64, i64, i64]
    L.oracle_nvfp4_quantize.restype = None
    L.oracle_nvfp4_quantize.argtypes = [u16p, i64, i64, i64, f32, u8p, u8p]
    L.oracle_sf_swizzled_offset.restype, L.oracle_sf_swizzled_offset.argtypes = i64, [i64, i64, i64]
    L.oracle_sf_swizzled_bytes.restype, L.oracle_sf_swizzled_bytes.argtypes = i64, [i64, i64]
    L.oracle_sf_swizzle.restype, L.oracle_sf_swizzle.argtypes = None, [u8p, i64, i64, u8p]
    L.oracle_nvfp4_dequantize.restype = None
    L.oracle_nvfp4_dequantize.argtypes = [u8p, u8p, f32, i64, i64, f64p]
    L.oracle_nvfp4_linear.restype = ctypes.c_int
    L.oracle_nvfp4_linear.argtypes = [u8p, u8p, f32, u8p, u8p, f32, u16p, i64, i64, i64p, i64, f64p]
    L.oracle_bf16_linear.restype = ctypes.c_int
    L.oracle_bf16_linear.argtypes = [u16p, i64, u16p, i64, u16p, i64, i64, i64p, i64, f64p]
    L.oracle_f64_to_bf16_array.restype, L.oracle_f64_to_bf16_array.argtypes = None, [f64p, i64, u16p]
    L.oracle_num_threads.restype, L.oracle_num_threads.argtypes = ctypes.c_int, []
    L.oracle_e8m0_decode.restype, L.oracle_e8m0_decode.argtypes = ctypes.c_double, [ctypes.c_uint8]
    L.oracle_mxfp4_quantize.restype, L.oracle_mxfp4_quantize.argtypes = None, [u16p, i64, i64, i64, u8p, u8p]
    L.oracle_mx_sf_swizzled_offset.restype, L.oracle_mx_sf_swizzled_offset.argtypes = i64, [i64, i64, i64]
    L.oracle_mx_sf_swizzled_bytes.restype, L.oracle_mx_sf_swizzled_bytes.argtypes = i64, [i64, i64]
    L.oracle_mx_sf_swizzle.restype, L.oracle_mx_sf_swizzle.argtypes = None, [u8p, i64, i64, u8p]
    L.oracle_mxfp4_dequantize.restype, L.oracle_mxfp4_dequantize.argtypes = None, [u8p, u8p, i64, i64, f64p]
    L.oracle_mxfp4_linear.restype = ctypes.c_int
    L.oracle_mxfp4_linear.argtypes = [u8p, u8p, u8p, u8p, u16p, i64, i64, i64p, i64, f64p]
    L.oracle_gelu_tanh.restype, L.oracle_gelu_tanh.argtypes = ctypes.c_double, [ctypes.c_double]
    L.oracle_gelu_tanh_array.restype, L.oracle_gelu_tanh_array.argtypes = None, [f64p, i64, f64p]
    L.oracle_layernorm_modulate.restype = None
    L.oracle_layernorm_modulate.argtypes = [u16p, i64, i64, i64, u16p, u16p, i64, ctypes.c_double, f64p]
    L.oracle_lora_merge.restype = None
    L.oracle_lora_merge.argtypes = [u16p, i64, u16p, i64, u16p, i64, i64, i64, i64, f32, u16p]
    _lib = L
    return L


def _p(a: np.ndarray, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {a.dtype}")
    return a


# ----------------------------------------------------------------- scalar codecs
def bf16_to_f32(h: int) -> float:
    return float(_load().oracle_bf16_to_f32(int(h)))


def f64_to_bf16(y: float) -> int:
    return int(_load().oracle_f64_to_bf16(float(y)))


def e2m1_decode(code: int) -> float:
    return float(_load().oracle_e2m1_decode(int(code)))


def e2m1_encode(y) -> int:
    return int(_load().oracle_e2m1_encode(np.float32(y)))


def e4m3_decode(code: int) -> float:
    return float(_load().oracle_e4m3_decode(int(code)))


def e4m3_encode(v) -> int:
    return int(_load().oracle_e4m3_encode(np.float32(v)))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


# ----------------------------------------------------------------- quantizer
def tensor_scale(x_bits: np.ndarray) -> np.float32:
    """T = amax(|x|) / 2688 as FP32 (1 for an all-zero tensor)."""
    x = _c(x_bits, np.uint16)
    rows, K = x.shape
    return np.float32(_load().oracle_tensor_scale(_p(x, ctypes.c_uint16), rows, K, K))


def quantize(x_bits: np.ndarray, T) -> tuple[np.ndarray, np.ndarray]:
    """BF16 bits [rows, K] -> (packed nibbles [rows, K/2], E4M3 scales [rows, K/16])."""
    x = _c(x_bits, np.uint16)
    rows, K = x.shape
    if K % 16:
        raise ValueError("K must be a multiple of 16")
    q = np.empty((rows, K // 2), np.uint8)
    sf = np.empty((rows, K // 16), np.uint8)
    _load().oracle_nvfp4_quantize(_p(x, ctypes.c_uint16), rows, K, K, np.float32(T),
                                  _p(q, ctypes.c_uint8), _p(sf, ctypes.c_uint8))
    return q, sf


def sf_swizzled_offset(r: int, kb: int, K: int) -> int:
    return int(_load().oracle_sf_swizzled_offset(r, kb, K))


def sf_swizzled_bytes(rows: int, K: int) -> int:
    return int(_load().oracle_sf_swizzled_bytes(rows, K))


def sf_swizzle(sf: np.ndarray, K: int) -> np.ndarray:
    """Row-major scales [rows, K/16] -> flat 128x4-chunked buffer (padding = 0)."""
    sf = _c(sf, np.uint8)
    rows = sf.shape[0]
    out = np.empty(sf_swizzled_bytes(rows, K), np.uint8)
    _load().oracle_sf_swizzle(_p(sf, ctypes.c_uint8), rows, K, _p(out, ctypes.c_uint8))
    return out


def dequantize(q: np.ndarray, sf: np.ndarray, T) -> np.ndarray:
    q, sf = _c(q, np.uint8), _c(sf, np.uint8)
    rows, K = q.shape[0], q.shape[1] * 2
    out = np.empty((rows, K), np.float64)
    _load().oracle_nvfp4_dequantize(_p(q, ctypes.c_uint8), _p(sf, ctypes.c_uint8), np.float32(T),
                                    rows, K, _p(out, ctypes.c_double))
    return out


# ----------------------------------------------------------------- matmuls
def _rows(rows, M):
    if rows is None:
        return None, M, None
    r = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    if r.size and (r.min() < 0 or r.max() >= M):
        raise IndexError("row index out of range")
    return r, int(r.size), _p(r, ctypes.c_int64)


def nvfp4_linear(qx, sfx, Tx, qw, sfw, Tw, bias_bits=None, rows=None) -> np.ndarray:
    """FP64 Y[rows, N] = dequant(X) @ dequant(W)^T + bias (the exact definition)."""
    qx, sfx, qw, sfw = _c(qx, np.uint8), _c(sfx, np.uint8), _c(qw, np.uint8), _c(sfw, np.uint8)
    M, K = qx.shape[0], qx.shape[1] * 2
    N = qw.shape[0]
    if qw.shape[1] * 2 != K:
        raise ValueError("K mismatch")
    keep, n_rows, rp = _rows(rows, M)
    b = None if bias_bits is None else _c(bias_bits, np.uint16)
    Y = np.empty((n_rows, N), np.float64)
    rc = _load().oracle_nvfp4_linear(_p(qx, ctypes.c_uint8), _p(sfx, ctypes.c_uint8), np.float32(Tx),
                                     _p(qw, ctypes.c_uint8), _p(sfw, ctypes.c_uint8), np.float32(Tw),
                                     None if b is None else _p(b, ctypes.c_uint16), N, K, rp, n_rows,
                                     _p(Y, ctypes.c_double))
    if rc:
        raise MemoryError("oracle_nvfp4_linear")
    del keep
    return Y


def bf16_linear(x_bits, w_bits, bias_bits=None, rows=None) -> np.ndarray:
    """FP64 Y[rows, N] = X @ W^T + bias on the raw BF16 values."""
    x, w = _c(x_bits, np.uint16), _c(w_bits, np.uint16)
    M, K = x.shape
    N = w.shape[0]
    if w.shape[1] != K:
        raise ValueError("K mismatch")
    keep, n_rows, rp = _rows(rows, M)
    b = None if bias_bits is None else _c(bias_bits, np.uint16)
    Y = np.empty((n_rows, N), np.float64)
    rc = _load().oracle_bf16_linear(_p(x, ctypes.c_uint16), K, _p(w, ctypes.c_uint16), K,
                                    None if b is None else _p(b, ctypes.c_uint16), N, K, rp, n_rows,
                                    _p(Y, ctypes.c_double))
    if rc:
        raise MemoryError("oracle_bf16_linear")
    del keep
    return Y


# ----------------------------------------------------------------- MXFP4
def e8m0_decode(b: int) -> float:
    return float(_load().oracle_e8m0_decode(int(b)))


def mxfp4_quantize(x_bits: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """BF16 bits [rows, K] -> (packed nibbles [rows, K/2], E8M0 scales [rows, K/32])."""
    x = _c(x_bits, np.uint16)
    rows, K = x.shape
    if K % 32:
        raise ValueError("K must be a multiple of 32")
    q = np.empty((rows, K // 2), np.uint8)
    sf = np.empty((rows, K // 32), np.uint8)
    _load().oracle_mxfp4_quantize(_p(x, ctypes.c_uint16), rows, K, K, _p(q, ctypes.c_uint8), _p(sf, ctypes.c_uint8))
    return q, sf


def mx_sf_swizzled_offset(r: int, kb: int, K: int) -> int:
    return int(_load().oracle_mx_sf_swizzled_offset(r, kb, K))


def mx_sf_swizzle(sf: np.ndarray, K: int) -> np.ndarray:
    sf = _c(sf, np.uint8)
    rows = sf.shape[0]
    out = np.empty(int(_load().oracle_mx_sf_swizzled_bytes(rows, K)), np.uint8)
    _load().oracle_mx_sf_swizzle(_p(sf, ctypes.c_uint8), rows, K, _p(out, ctypes.c_uint8))
    return out


def mxfp4_dequantize(q: np.ndarray, sf: np.ndarray) -> np.ndarray:
    q, sf = _c(q, np.uint8), _c(sf, np.uint8)
    rows, K = q.shape[0], q.shape[1] * 2
    out = np.empty((rows, K), np.float64)
    _load().oracle_mxfp4_dequantize(_p(q, ctypes.c_uint8), _p(sf, ctypes.c_uint8), rows, K, _p(out, ctypes.c_double))
    return out


def mxfp4_linear(qx, sfx, qw, sfw, bias_bits=None, rows=None) -> np.ndarray:
    """Y = dequant(X) . dequant(W)^T + bias in FP64 for `rows` of X (all rows when None)."""
    qx, sfx, qw, sfw = _c(qx, np.uint8), _c(sfx, np.uint8), _c(qw, np.uint8), _c(sfw, np.uint8)
    M, K = qx.shape[0], qx.shape[1] * 2
    N = qw.shape[0]
    if qw.shape[1] * 2 != K:
        raise ValueError("K mismatch")
    keep, n_rows, rp = _rows(rows, M)
    Y = np.empty((n_rows, N), np.float64)
    b = _c(bias_bits, np.uint16) if bias_bits is not None else None
    rc = _load().oracle_mxfp4_linear(_p(qx, ctypes.c_uint8), _p(sfx, ctypes.c_uint8), _p(qw, ctypes.c_uint8),
                                     _p(sfw, ctypes.c_uint8), _p(b, ctypes.c_uint16) if b is not None else None,
                                     N, K, rp, n_rows, _p(Y, ctypes.c_double))
    if rc:
        raise MemoryError("oracle_mxfp4_linear")
    del keep
    return Y


# ----------------------------------------------------------------- linear with quantized output
ACT_NONE, ACT_GELU_TANH = 0, 1


def gelu_tanh(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty_like(x)
    _load().oracle_gelu_tanh_array(_p(x, ctypes.c_double), x.size, _p(out, ctypes.c_double))
    return out


def nvfp4_linear_quantized(qx, sfx, Tx, qw, sfw, Tw, bias_bits, act: int, T_out, rows=None):
    """The NVFP4 linear followed by an activation and the activation quantizer of the NEXT linear.

    H = act(Y) with Y the FP64 linear; h = H rounded once to BF16 (what an unfused pipeline would
    store); (q, sf) = quantize(h, T_out) with a caller-supplied T_out.  Returns (H as FP64, h bits,
    packed nibbles, row-major scales).
    """
    Y = nvfp4_linear(qx, sfx, Tx, qw, sfw, Tw, bias_bits, rows=rows)
    H = gelu_tanh(Y) if act == ACT_GELU_TANH else Y
    h = round_bf16(H)
    q, sf = quantize(h, T_out)
    return H, h, q, sf


def mxfp4_linear_quantized(qx, sfx, qw, sfw, bias_bits, act: int, rows=None):
    """The MXFP4 linear followed by an activation and the MXFP4 quantizer of the NEXT linear: H = act(Y),
    h = H rounded once to BF16, (q, sf) = mxfp4_quantize(h).  Returns (H as FP64, h bits, nibbles, row-major scales)."""
    Y = mxfp4_linear(qx, sfx, qw, sfw, bias_bits, rows=rows)
    H = gelu_tanh(Y) if act == ACT_GELU_TANH else Y
    h = round_bf16(H)
    q, sf = mxfp4_quantize(h)
    return H, h, q, sf


LN_EPS = 1e-6


def layernorm_modulate(x_bits, scale_bits, shift_bits, rows_per_sample: int, eps: float = LN_EPS) -> np.ndarray:
    """FP64 y = LN(x) * (1 + scale[sample]) + shift[sample]; x [rows, K], scale/shift [samples, K] BF16 bits."""
    x, sc, sh = _c(x_bits, np.uint16), _c(scale_bits, np.uint16), _c(shift_bits, np.uint16)
    rows, K = x.shape
    samples = (rows + rows_per_sample - 1) // rows_per_sample
    if sc.shape != (samples, K) or sh.shape != (samples, K):
        raise ValueError("scale/shift must be [samples, K]")
    out = np.empty((rows, K), np.float64)
    _load().oracle_layernorm_modulate(_p(x, ctypes.c_uint16), rows, K, K, _p(sc, ctypes.c_uint16),
                                      _p(sh, ctypes.c_uint16), rows_per_sample, float(eps), _p(out, ctypes.c_double))
    return out


def layernorm_modulate_quantized(x_bits, scale_bits, shift_bits, rows_per_sample: int, T, eps: float = LN_EPS):
    """(Y FP64, h = bf16(Y) bits, nibbles, row-major scales): the normalised input of a linear, quantized."""
    Y = layernorm_modulate(x_bits, scale_bits, shift_bits, rows_per_sample, eps)
    h = round_bf16(Y)
    q, sf = quantize(h, T)
    return Y, h, q, sf


# ----------------------------------------------------------------- weight refresh
def lora_merge(w_bits: np.ndarray, a_bits: np.ndarray, b_bits: np.ndarray, scaling) -> np.ndarray:
    """W' = bf16(W + s * B A) in the fixed binary32 order; W [N, K], A [r, K], B [N, r] as BF16 bits."""
    w, a, b = _c(w_bits, np.uint16), _c(a_bits, np.uint16), _c(b_bits, np.uint16)
    N, K = w.shape
    r = a.shape[0]
    if a.shape != (r, K) or b.shape != (N, r):
        raise ValueError("shapes: W [N, K], A [r, K], B [N, r]")
    out = np.empty((N, K), np.uint16)
    _load().oracle_lora_merge(_p(w, ctypes.c_uint16), K, _p(a, ctypes.c_uint16), K, _p(b, ctypes.c_uint16), r,
                              N, K, r, np.float32(scaling), _p(out, ctypes.c_uint16))
    return out


def requantize_lora(w_bits, a_bits, b_bits, scaling):
    """Merge, then the weight quantizer: (W' bits, packed nibbles, row-major scales, T)."""
    merged = lora_merge(w_bits, a_bits, b_bits, scaling)
    T = tensor_scale(merged)
    q, sf = quantize(merged, T)
    return merged, q, sf, T


def round_bf16(y: np.ndarray) -> np.ndarray:
    """One nearest-even rounding of FP64 values to BF16 bit patterns."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    out = np.empty(y.shape, np.uint16)
    _load().oracle_f64_to_bf16_array(_p(y, ctypes.c_double), y.size, _p(out, ctypes.c_uint16))
    return out


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """BF16 bit patterns -> their exact values as FP64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def linear_tolerance(Y: np.ndarray) -> np.ndarray:
    """Per-output bound 2^-7 |Y| + 1e-4 rms(Y[row, :]) that a GPU result must meet."""
    rms = np.sqrt(np.mean(Y * Y, axis=1, keepdims=True))
    return 2.0 ** -7 * np.abs(Y) + 1e-4 * rms
