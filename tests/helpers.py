"""Shared helpers for the GPU parity tests (host-side glue only)."""
import numpy as np
import torch

import oracle


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(bits: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(device)


def swizzled_offsets(rows: np.ndarray, K: int) -> np.ndarray:
    """[len(rows), K/16] byte offsets into the 128x4-chunked scale buffer (vectorised copy of the
    index rule; checked against the oracle's scalar function in the tests)."""
    nb = K // 16
    chunks_k = (nb + 3) // 4
    r = np.asarray(rows, dtype=np.int64)[:, None]
    b = np.arange(nb, dtype=np.int64)[None, :]
    rr = r % 128
    return ((r // 128) * chunks_k + b // 4) * 512 + (rr % 32) * 16 + (rr // 32) * 4 + b % 4


def unswizzle_rows(sf_swizzled: np.ndarray, rows, K: int) -> np.ndarray:
    return sf_swizzled[swizzled_offsets(rows, K)]


def sample_rows(M: int, seed: int = 0) -> np.ndarray:
    """First and last 128-row tile in full plus one pseudo-random row of every other tile."""
    from paper_2604_06916_b200 import workloads
    return workloads.sample_rows(M, seed)


def check_linear(y_gpu_bits: np.ndarray, Y: np.ndarray, what: str = ""):
    """|gpu - oracle| <= 2^-7 |oracle| + 1e-4 rms(oracle row) for every output."""
    g = oracle.bits_to_f64(y_gpu_bits)
    tol = oracle.linear_tolerance(Y)
    err = np.abs(g - Y)
    bad = err > tol
    if bad.any():
        i, j = np.argwhere(bad)[0]
        raise AssertionError(
            f"{what}: {int(bad.sum())} of {bad.size} outputs out of tolerance; first at ({i},{j}): "
            f"gpu={g[i, j]!r} oracle={Y[i, j]!r} err={err[i, j]:.3e} tol={tol[i, j]:.3e}; "
            f"bad rows={np.unique(np.argwhere(bad)[:, 0])[:8]} bad cols={np.unique(np.argwhere(bad)[:, 1])[:8]}")
    return float(np.max(err / np.maximum(tol, 1e-300)))


def dequantize_on_device(q: torch.Tensor, sf_swizzled: torch.Tensor, rows: int, K: int) -> torch.Tensor:
    """code * block scale as BF16 (exact: at most 6 significant bits), built from plain torch ops.

    A secondary, full-coverage screen for the GEMMs; the tensor scale is left out so that every
    value is representable.  The swizzled-scale index rule is the vectorised copy checked against
    the oracle's scalar function.
    """
    dev = q.device
    lut = torch.tensor([0, .5, 1, 1.5, 2, 3, 4, 6, -0., -.5, -1, -1.5, -2, -3, -4, -6], dtype=torch.float32, device=dev)
    lo = lut[(q & 0xF).long()]
    hi = lut[(q >> 4).long()]
    vals = torch.stack((lo, hi), dim=-1).reshape(rows, K)
    offs = torch.from_numpy(swizzled_offsets(np.arange(rows), K)).to(dev)
    sb = sf_swizzled.reshape(-1)[offs].to(torch.int32)
    e, m = (sb >> 3) & 15, sb & 7
    scale = torch.where(e == 0, m.float() * 2.0 ** -9, torch.ldexp(1.0 + m.float() / 8.0, e - 7))
    out = (vals.reshape(rows, K // 16, 16) * scale[:, :, None]).reshape(rows, K)
    out_bf16 = out.to(torch.bfloat16)
    assert torch.equal(out_bf16.float(), out)
    return out_bf16
