"""Pins for the oracle's stage-1 selection and rank-consistency metrics -- CPU only."""
import itertools

import numpy as np
import scipy.stats

from oracle import selection as S


def test_selection_brute_force_all_orderings_of_six():
    vals = np.array([0.5, -1.0, 2.0, 3.5, 0.0, -2.5])
    for perm in itertools.permutations(range(6)):
        r = vals[list(perm)]
        got = S.select_contrastive(r[None, :], 4)[0]
        best = [i for i in range(6) if r[i] in (3.5, 2.0)]
        worst = [i for i in range(6) if r[i] in (-2.5, -1.0)]
        assert set(got[:2]) == set(best) and set(got[2:]) == set(worst)
        assert r[got[0]] == 3.5 and r[got[1]] == 2.0 and r[got[2]] == -2.5 and r[got[3]] == -1.0


def test_ties_go_to_the_lower_index_and_full_selection_is_a_permutation():
    r = np.array([[1.0, 3.0, 3.0, 0.0, 0.0, 3.0, 1.0, 0.0]])
    assert list(S.descending_ranks(r[0])) == [3, 0, 1, 5, 6, 2, 4, 7]
    got = S.select_contrastive(r, 4)[0]
    assert list(got) == [1, 2, 7, 4]
    full = S.select_contrastive(r, 8)[0]
    assert sorted(full) == list(range(8))


def test_selection_invariant_under_increasing_affine_maps_and_mirrored_under_negation():
    rng = np.random.default_rng(0)
    r = rng.standard_normal((7, 96))
    a = S.select_contrastive(r, 24)
    assert np.array_equal(a, S.select_contrastive(3.0 * r - 11.0, 24))
    b = S.select_contrastive(-r, 24)
    assert np.array_equal(a[:, :12], b[:, 12:]) and np.array_equal(a[:, 12:], b[:, :12])


def test_selected_range_never_loses_more_than_four_delta():
    # the inequality behind the extreme-value guarantee: with |eps_i| <= Delta, the true range of the
    # candidates picked on the proxy rewards is at least the true range minus 4 Delta, trial by trial
    rng = np.random.default_rng(1)
    N, delta, sigma = 96, 0.3, 1.0
    R = rng.standard_normal((2000, N)) * sigma
    proxy = R + rng.uniform(-delta, delta, size=R.shape)
    sel = S.select_contrastive(proxy, 2)
    rows = np.arange(R.shape[0])
    w_hat = R[rows, sel[:, 0]] - R[rows, sel[:, 1]]
    w_star = R.max(axis=1) - R.min(axis=1)
    assert np.all(w_hat >= w_star - 4 * delta - 1e-12)
    # E[W*] approaches 2 sigma sqrt(2 log N) from below; at N = 96 the ratio is about 0.83
    ratio = w_star.mean() / (2 * sigma * np.sqrt(2 * np.log(N)))
    assert 0.78 < ratio < 0.88
    R2 = rng.standard_normal((2000, 4 * N)) * sigma
    assert (R2.max(axis=1) - R2.min(axis=1)).mean() > w_star.mean()          # the range grows with N


def test_advantages_are_standardised_with_the_population_deviation():
    rng = np.random.default_rng(2)
    r = rng.standard_normal((5, 96)) * 3 + 7
    A = S.group_advantages(r)
    assert np.allclose(A.mean(axis=1), 0, atol=1e-13) and np.allclose((A ** 2).mean(axis=1), 1, atol=1e-12)
    assert np.allclose(A, scipy.stats.zscore(r, axis=1, ddof=0), atol=1e-12)      # library routine
    assert np.allclose(S.group_advantages(np.array([[1.0, 3.0]])), [[-1.0, 1.0]])
    assert np.array_equal(S.group_advantages(np.full((1, 8), 2.5)), np.zeros((1, 8)))


def test_rank_metrics_against_scipy_and_closed_forms():
    rng = np.random.default_rng(3)
    ref = rng.standard_normal((6, 40))
    proxy = ref + 0.3 * rng.standard_normal((6, 40))
    ints, fl = S.rank_consistency(ref, proxy, 4)
    for p in range(6):
        assert abs(fl[p, 0] - scipy.stats.kendalltau(ref[p], proxy[p]).statistic) < 1e-12   # no ties: tau-a = tau-b
        assert abs(fl[p, 1] - scipy.stats.spearmanr(ref[p], proxy[p]).statistic) < 1e-12
        top_ref, top_px = set(np.argsort(-ref[p])[:4]), set(np.argsort(-proxy[p])[:4])
        bot_ref, bot_px = set(np.argsort(ref[p])[:4]), set(np.argsort(proxy[p])[:4])
        assert ints[p, 2] == len(top_ref & top_px) and ints[p, 3] == len(bot_ref & bot_px)
    same, _ = S.rank_consistency(ref, ref, 4)
    assert np.all(same[:, 0] == 40 * 39 // 2) and np.all(same[:, 1] == 0) and np.all(same[:, 2:] == 4)
    _, rev = S.rank_consistency(ref, -ref, 4)
    assert np.allclose(rev[:, 0], -1) and np.allclose(rev[:, 1], -1) and np.all(rev[:, 2:] == 0)
    # hand-worked: ref ranks 0,1,2,3 against proxy ranks 1,0,2,3: one discordant pair of six, d^2 = 2
    ints, fl = S.rank_consistency(np.array([[4.0, 3.0, 2.0, 1.0]]), np.array([[3.0, 4.0, 2.0, 1.0]]), 1)
    assert list(ints[0]) == [4, 2, 0, 1] and abs(fl[0, 0] - 4 / 6) < 1e-15 and abs(fl[0, 1] - 0.8) < 1e-15
