"""Pins for the oracle's GELU and for the linear-with-quantized-output composition -- CPU only."""
import numpy as np
import torch

import oracle


def test_gelu_against_library_routine_in_fp64():
    x = np.concatenate([np.linspace(-12, 12, 4001), np.random.default_rng(0).standard_normal(2000) * 3])
    want = torch.nn.functional.gelu(torch.from_numpy(x), approximate="tanh").numpy()
    assert np.max(np.abs(oracle.gelu_tanh(x) - want)) <= 1e-14 * np.maximum(1.0, np.abs(want)).max()


def test_gelu_closed_form_properties():
    x = np.linspace(-8, 8, 1601)
    g = oracle.gelu_tanh(x)
    # x/2 (1 + tanh u) - (-x/2)(1 + tanh(-u)) = x: the odd part of gelu is x/2
    assert np.max(np.abs(g - oracle.gelu_tanh(-x) - x)) < 1e-14
    assert oracle.gelu_tanh(np.array([0.0]))[0] == 0.0
    assert abs(oracle.gelu_tanh(np.array([30.0]))[0] - 30.0) < 1e-12     # identity far right
    assert abs(oracle.gelu_tanh(np.array([-30.0]))[0]) < 1e-12           # zero far left
    h = 1e-6
    slope = (oracle.gelu_tanh(np.array([h]))[0] - oracle.gelu_tanh(np.array([-h]))[0]) / (2 * h)
    assert abs(slope - 0.5) < 1e-9                                        # gelu'(0) = 1/2
    # between x * Phi bounds: 0 <= gelu(x) <= x for x >= 0, and -0.2 < gelu(x) <= 0 for x <= 0
    assert np.all(g[x >= 0] >= 0) and np.all(g[x >= 0] <= x[x >= 0] + 1e-15)
    assert np.all(g[x <= 0] <= 1e-300) and np.all(g[x <= 0] > -0.2)
    # the constant inside is sqrt(2/pi): with u = c x (1 + 0.044715 x^2), tanh(u) = 2 g / x - 1
    xs = np.array([0.5, 1.0, 2.0])
    u = np.arctanh(2 * oracle.gelu_tanh(xs) / xs - 1)
    assert np.allclose(u / (xs * (1 + 0.044715 * xs ** 2)), np.sqrt(2 / np.pi), rtol=1e-12)


def test_quantized_output_is_the_composition_of_pinned_parts():
    rng = np.random.default_rng(3)
    M, N, K = 8, 32, 64
    xb = (torch.from_numpy(rng.standard_normal((M, K))).to(torch.bfloat16)).view(torch.int16).numpy().view(np.uint16)
    wb = (torch.from_numpy(rng.standard_normal((N, K)) * 0.2).to(torch.bfloat16)).view(torch.int16).numpy().view(np.uint16)
    Tx, Tw = oracle.tensor_scale(xb), oracle.tensor_scale(wb)
    qx, sfx = oracle.quantize(xb, Tx)
    qw, sfw = oracle.quantize(wb, Tw)
    for act in (oracle.ACT_NONE, oracle.ACT_GELU_TANH):
        H, h, q, sf = oracle.nvfp4_linear_quantized(qx, sfx, Tx, qw, sfw, Tw, None, act, 0.01)
        Y = oracle.nvfp4_linear(qx, sfx, Tx, qw, sfw, Tw)
        want_H = Y if act == oracle.ACT_NONE else torch.nn.functional.gelu(torch.from_numpy(Y), approximate="tanh").numpy()
        assert np.allclose(H, want_H, rtol=0, atol=1e-13)
        assert np.array_equal(h, oracle.round_bf16(H))
        q2, sf2 = oracle.quantize(h, 0.01)
        assert np.array_equal(q, q2) and np.array_equal(sf, sf2)


def _bits(t):
    return t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_layernorm_modulate_against_library_routine_and_invariants():
    rng = np.random.default_rng(7)
    rows, K, rps = 12, 96, 4
    x = torch.from_numpy(rng.standard_normal((rows, K)) * 3 + 1.5).to(torch.bfloat16)
    sc = torch.from_numpy(rng.standard_normal((3, K)) * 0.2).to(torch.bfloat16)
    sh = torch.from_numpy(rng.standard_normal((3, K)) * 0.1).to(torch.bfloat16)
    Y = oracle.layernorm_modulate(_bits(x), _bits(sc), _bits(sh), rps)
    xd, scd, shd = x.double(), sc.double(), sh.double()
    ln = torch.nn.functional.layer_norm(xd, (K,), eps=oracle.LN_EPS)                    # library routine, FP64
    want = ln * (1 + scd.repeat_interleave(rps, dim=0)) + shd.repeat_interleave(rps, dim=0)
    assert np.max(np.abs(Y - want.numpy())) < 1e-12
    # zero modulation: rows have mean 0 and variance var / (var + eps)
    z = torch.zeros((3, K), dtype=torch.bfloat16)
    Y0 = oracle.layernorm_modulate(_bits(x), _bits(z), _bits(z), rps)
    var = xd.var(dim=1, unbiased=False).numpy()
    assert np.allclose(Y0.mean(axis=1), 0, atol=1e-13) and np.allclose((Y0 ** 2).mean(axis=1), var / (var + oracle.LN_EPS))
    # invariant under a*x + b of the input (a > 0, up to eps) -- powers of two keep the inputs exact in BF16
    Y4 = oracle.layernorm_modulate(_bits(x * 4), _bits(z), _bits(z), rps)
    assert np.max(np.abs(Y4 - Y0)) < 1e-6
    # the sample index really selects the modulation row: rows 4..7 use scale[1]
    sc2 = torch.zeros((3, K), dtype=torch.bfloat16)
    sc2[1] = 1.0
    Y2 = oracle.layernorm_modulate(_bits(x), _bits(sc2), _bits(z), rps)
    assert np.allclose(Y2[4:8], 2 * Y0[4:8]) and np.allclose(Y2[:4], Y0[:4]) and np.allclose(Y2[8:], Y0[8:])
    # constant row: xhat = 0, output = shift
    xc = torch.full((4, K), 2.5, dtype=torch.bfloat16)
    Yc = oracle.layernorm_modulate(_bits(xc), _bits(sc[:1]), _bits(sh[:1]), 4)
    assert np.allclose(Yc, sh[:1].double().numpy().repeat(4, axis=0))
