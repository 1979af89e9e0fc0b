"""Pins for the attention oracle -- CPU only.  None of them re-types its formula: closed forms,
a hand-worked case, invariances, and a library routine (torch's scaled-dot-product attention in FP64)."""
import math

import numpy as np
import torch

from oracle import attention as A


def rnd(rng, *shape, scale=1.0):
    t = torch.from_numpy(rng.standard_normal(shape) * scale).to(torch.bfloat16)
    return t.to(torch.float64).numpy()


def test_single_key_returns_its_value():
    rng = np.random.default_rng(0)
    q, k, v = rnd(rng, 5, 16), rnd(rng, 1, 16), rnd(rng, 1, 16)
    assert np.array_equal(A.attention_head(q, k, v), np.repeat(v, 5, axis=0))


def test_equal_keys_give_the_mean_of_the_values():
    rng = np.random.default_rng(1)
    q, v = rnd(rng, 7, 32), rnd(rng, 9, 32)
    k = np.repeat(rnd(rng, 1, 32), 9, axis=0)
    np.testing.assert_allclose(A.attention_head(q, k, v), np.repeat(v.mean(0, keepdims=True), 7, 0), rtol=1e-14)


def test_two_keys_by_hand():
    # d = 4, q = (2,0,0,0); k0 = 0, k1 = (ln 3, 0,0,0): scores 0 and 2 ln3 / sqrt(4) = ln 3 -> weights 1/4, 3/4
    q = np.array([[2.0, 0, 0, 0]])
    k = np.array([[0.0, 0, 0, 0], [math.log(3.0), 0, 0, 0]])
    v = np.array([[4.0, 0, 8, -4], [0.0, 4, 0, 4]])
    np.testing.assert_allclose(A.attention_head(q, k, v), [[1.0, 3.0, 2.0, 2.0]], rtol=1e-15)


def test_scale_is_one_over_sqrt_d_not_d():
    # d = 16: q.k = 16 ln 2 / ... choose q = 4 e0, k1 = ln2 e0: score = 4 ln2 / 4 = ln 2 -> weights 1/3, 2/3
    q = np.zeros((1, 16)); q[0, 0] = 4.0
    k = np.zeros((2, 16)); k[1, 0] = math.log(2.0)
    v = np.zeros((2, 16)); v[0, 0] = 3.0; v[1, 1] = 3.0
    out = A.attention_head(q, k, v)
    np.testing.assert_allclose(out[0, :2], [1.0, 2.0], rtol=1e-15)


def test_dominant_key_selects_its_value():
    rng = np.random.default_rng(2)
    q, k, v = rnd(rng, 4, 64), rnd(rng, 33, 64, scale=0.01), rnd(rng, 33, 64)
    k[17] = q[2] * 100.0           # query 2 scores this key far above the rest
    out = A.attention_head(q, k, v)
    np.testing.assert_allclose(out[2], v[17], atol=1e-12)


def test_invariant_to_key_order_and_to_a_common_key_shift():
    rng = np.random.default_rng(3)
    q, k, v = rnd(rng, 6, 32), rnd(rng, 50, 32), rnd(rng, 50, 32)
    ref = A.attention_head(q, k, v)
    perm = rng.permutation(50)
    np.testing.assert_allclose(A.attention_head(q, k[perm], v[perm]), ref, rtol=1e-12, atol=1e-14)
    # adding the same vector to every key adds a per-query constant to the scores
    np.testing.assert_allclose(A.attention_head(q, k + rnd(rng, 1, 32), v), ref, rtol=1e-10, atol=1e-12)


def test_output_is_a_convex_combination():
    rng = np.random.default_rng(4)
    q, k, v = rnd(rng, 20, 32, scale=3.0), rnd(rng, 70, 32, scale=3.0), rnd(rng, 70, 32)
    out = A.attention_head(q, k, v)
    assert np.all(out <= v.max(0) + 1e-12) and np.all(out >= v.min(0) - 1e-12)
    # and of constant values it is that constant
    np.testing.assert_allclose(A.attention_head(q, k, np.full((70, 32), 0.75)), 0.75, rtol=1e-14)


def test_against_the_library_routine_in_fp64():
    rng = np.random.default_rng(5)
    B, Sq, Skv, H, d = 2, 37, 91, 3, 128
    q, k, v = rnd(rng, B, Sq, H, d), rnd(rng, B, Skv, H, d), rnd(rng, B, Skv, H, d)
    tq, tk, tv = (torch.from_numpy(a).permute(0, 2, 1, 3) for a in (q, k, v))     # [B, H, S, d]
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    np.testing.assert_allclose(A.attention(q, k, v), want, rtol=1e-12, atol=1e-14)
    rows = [0, 5, 36]
    np.testing.assert_allclose(A.attention(q, k, v, rows=rows), want[:, rows], rtol=1e-12, atol=1e-14)


def test_large_scores_do_not_overflow():
    q = np.full((1, 128), 30.0); k = np.stack([np.full(128, 30.0), np.full(128, -30.0)]); v = np.array([[1.0] * 128, [5.0] * 128])
    out = A.attention_head(q, k, v)    # scores +-1.15e5 / 11.3: exp of the raw score overflows FP64
    assert np.all(np.isfinite(out)) and np.allclose(out, 1.0)


def test_joint_streams_are_the_concatenation():
    rng = np.random.default_rng(6)
    a = tuple(rnd(rng, 2, 8, 2, 16) for _ in range(3))
    b = tuple(rnd(rng, 2, 5, 2, 16) for _ in range(3))
    oa, ob = A.attention_joint(a, b)
    # every query of either stream sees all 13 keys: with the second stream's values set to a constant c and
    # the first's to 0 the output is c times the probability mass on the second stream, the same for both halves
    a0 = (a[0], a[1], np.zeros_like(a[2]))
    b1 = (b[0], b[1], np.ones_like(b[2]))
    ma, mb = A.attention_joint(a0, b1)
    assert np.all((ma > 0) & (ma < 1)) and np.all((mb > 0) & (mb < 1))
    # and a single stream split in two gives back the single-stream result
    q, k, v = (np.concatenate((x, y), axis=1) for x, y in zip(a, b))
    whole = A.attention(q, k, v)
    np.testing.assert_array_equal(np.concatenate((oa, ob), axis=1), whole)
