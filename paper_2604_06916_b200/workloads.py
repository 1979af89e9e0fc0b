"""Seeded synthetic inputs shaped like the diffusion-transformer linears of the rollout.

This module holds generators and shape tables only -- none of the quantizer or
matmul arithmetic -- so both the CUDA tests and the CPU oracle tests can draw the
same tensors from it.  Trained FLUX.1 / SD3.5-Large / SANA weights and real
activations are not available; these distributions stand in for them:

* ``outlier``   N(0,1) with 0.5 % of entries multiplied by 20
* ``channel``   N(0,1) times a per-input-channel scale, log-uniform in [0.1, 10]
* ``student_t`` heavy-tailed Student-t with 3 degrees of freedom

Weights are N(0, sigma) with sigma = 0.02 (config 1) or 1/sqrt(K); biases N(0, 0.01).
Draw order per layer: X, (channel scales), W, bias, from one ``torch.Generator``
seeded with ``seed * 1000 + layer_index`` on the device asked for.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Layer:
    name: str
    M: int
    K: int
    N: int


@dataclass(frozen=True)
class Config:
    name: str
    seed: int
    activation: str  # "outlier" | "channel" | "student_t"
    weight_sigma: float | None  # None -> 1/sqrt(K)
    layers: tuple[Layer, ...]


def _mk(name, seed, act, wsig, M, shapes):
    return Config(name, seed, act, wsig, tuple(Layer(n, M, k, nn) for n, k, nn in shapes))


CONFIG_SINGLE = _mk("single", 0, "outlier", 0.02, 256, [("lin", 512, 512)])
CONFIG_SANA = _mk("sana_1p6b_g16", 1, "channel", None, 1024 * 16,
                  [("qkv", 2240, 6720), ("attn_out", 2240, 2240), ("ffn_in", 2240, 5600),
                   ("ffn_out", 5600, 2240)])
CONFIG_SD35 = _mk("sd35_large_g8", 2, "channel", None, (4096 + 333) * 8,
                  [("qkv", 2432, 7296), ("out", 2432, 2432), ("mlp_in", 2432, 9728),
                   ("mlp_out", 9728, 2432)])
CONFIG_FLUX = _mk("flux1_12b_g8", 3, "student_t", None, (4096 + 512) * 8,
                  [("d_qkv", 3072, 9216), ("d_proj", 3072, 3072), ("d_mlp_in", 3072, 12288),
                   ("d_mlp_out", 12288, 3072), ("s_fused", 3072, 21504), ("s_out", 15360, 3072)])

# the geometry the paper trained FLUX.1 at (512 x 512 images: 1024 image + 512 text tokens), same layers
CONFIG_FLUX_512 = _mk("flux1_12b_512px_g8", 5, "student_t", None, (1024 + 512) * 8,
                      [("d_qkv", 3072, 9216), ("d_proj", 3072, 3072), ("d_mlp_in", 3072, 12288),
                       ("d_mlp_out", 12288, 3072), ("s_fused", 3072, 21504), ("s_out", 15360, 3072)])

SWEEP_GROUPS = (4, 8, 16, 32, 64)
SWEEP_TOKENS = 4608
SWEEP_STEPS = 28


def config_sweep(group: int) -> Config:
    """Rollout-scaling sweep: the FLUX single-stream pair at a given group size."""
    return _mk(f"flux1_sweep_g{group}", 4, "student_t", None, SWEEP_TOKENS * group,
               [("s_fused", 3072, 21504), ("s_out", 15360, 3072)])


CONFIGS = {c.name: c for c in (CONFIG_SINGLE, CONFIG_SANA, CONFIG_SD35, CONFIG_FLUX, CONFIG_FLUX_512)}


def _normal(shape, gen, device, chunk_rows=4096):
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)


def make_activation(kind: str, M: int, K: int, gen: torch.Generator, device) -> torch.Tensor:
    """bf16 [M, K]; generated in row chunks so the FP32 temporaries stay small."""
    out = torch.empty((M, K), dtype=torch.bfloat16, device=device)
    scale = None
    if kind == "channel":
        u = torch.rand((K,), generator=gen, device=device, dtype=torch.float32) * 2.0 - 1.0
        scale = torch.pow(torch.tensor(10.0, device=device), u)
    rows_per_chunk = max(1, (1 << 25) // K)
    for r0 in range(0, M, rows_per_chunk):
        r1 = min(M, r0 + rows_per_chunk)
        z = _normal((r1 - r0, K), gen, device)
        if kind == "outlier":
            mask = torch.rand((r1 - r0, K), generator=gen, device=device) < 0.005
            z = torch.where(mask, z * 20.0, z)
        elif kind == "channel":
            z = z * scale
        elif kind == "student_t":
            d = _normal((r1 - r0, K), gen, device).square_()
            d += _normal((r1 - r0, K), gen, device).square_()
            d += _normal((r1 - r0, K), gen, device).square_()
            z = z / torch.sqrt(d / 3.0)
        else:
            raise ValueError(kind)
        out[r0:r1] = z.to(torch.bfloat16)
    return out


def make_layer(cfg: Config, index: int, device="cpu", M: int | None = None, with_bias: bool = True):
    """Returns (X bf16 [M,K], W bf16 [N,K], bias bf16 [N] or None) for cfg.layers[index].

    ``M`` overrides the row count (tests use a slice of the full problem).
    """
    layer = cfg.layers[index]
    rows = layer.M if M is None else M
    gen = torch.Generator(device=device)
    gen.manual_seed(cfg.seed * 1000 + index)
    X = make_activation(cfg.activation, rows, layer.K, gen, device)
    sigma = cfg.weight_sigma if cfg.weight_sigma is not None else layer.K ** -0.5
    W = torch.empty((layer.N, layer.K), dtype=torch.bfloat16, device=device)
    rows_per_chunk = max(1, (1 << 25) // layer.K)
    for r0 in range(0, layer.N, rows_per_chunk):
        r1 = min(layer.N, r0 + rows_per_chunk)
        W[r0:r1] = (_normal((r1 - r0, layer.K), gen, device) * sigma).to(torch.bfloat16)
    bias = None
    if with_bias:
        bias = (_normal((layer.N,), gen, device) * 0.01).to(torch.bfloat16)
    return X, W, bias


LORA_RANK = 32    # Section 4.1: rank 32, alpha 64 in every experiment
LORA_ALPHA = 64.0


def make_lora(N: int, K: int, seed: int, device="cpu", rank: int = LORA_RANK):
    """Adapter factors of a trained policy, (A bf16 [rank, K], B bf16 [N, rank]).

    A keeps its Gaussian init (sigma = 1/rank, the usual default); B starts at zero and drifts
    during training, modelled as N(0, 0.02^2) so that (alpha/rank) * B A perturbs a weight of
    sigma K^-1/2 by a few per cent and moves most of its BF16 bits.
    """
    gen = torch.Generator(device=device)
    gen.manual_seed(77_000 + seed)
    A = (_normal((rank, K), gen, device) * (1.0 / rank)).to(torch.bfloat16)
    B = (_normal((N, rank), gen, device) * 0.02).to(torch.bfloat16)
    return A, B


def make_qkv(batch: int, seq: int, heads: int, seed: int, device="cpu", q_gain: float = 1.0, head_dim: int = 128):
    """One fused projection output [batch, seq, 3 * heads * head_dim] in BF16 and its q, k, v views.

    q and k are unit normal per element (the models named in Section 4.1 RMS-normalise both per head
    before attention, so q.k / sqrt(d) has unit variance); v is normal with standard deviation 0.5.
    `q_gain` > 1 sharpens the softmax.  The views are [batch, seq, heads, head_dim] with a token pitch of
    3 * heads * head_dim elements, as attention sees them after a fused q/k/v linear.
    """
    g = torch.Generator(device=device).manual_seed(7000 + seed)
    width = heads * head_dim
    fused = torch.empty((batch, seq, 3 * width), dtype=torch.bfloat16, device=device)
    for b in range(batch):
        z = torch.randn((seq, 3 * width), generator=g, device=device, dtype=torch.float32)
        z[:, :width] *= q_gain
        z[:, 2 * width:] *= 0.5
        fused[b] = z.to(torch.bfloat16)
    q, k, v = (fused[:, :, i * width:(i + 1) * width].unflatten(2, (heads, head_dim)) for i in range(3))
    return fused, q, k, v


def sample_rows(M: int, seed: int = 0):
    """Row sample of an [M, ...] problem used wherever the CPU oracle cannot afford every row: the first and
    the last 128-row tile in full plus one pseudo-random row of every other tile (numpy int64, sorted)."""
    import numpy as np

    rng = np.random.default_rng(seed)
    tiles = (M + 127) // 128
    rows = set(range(min(128, M))) | set(range((tiles - 1) * 128, M))
    for t in range(1, tiles - 1):
        rows.add(t * 128 + int(rng.integers(0, 128)))
    return np.array(sorted(rows), dtype=np.int64)


def to_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    import numpy as np

    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
