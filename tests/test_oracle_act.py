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
