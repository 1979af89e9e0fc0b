"""TEST INFRASTRUCTURE -- plain CPU statement of the stage-1 selection step and of the
rank-consistency metrics; shares nothing with the CUDA path.

Section 3.4 / Section 4.1 ("Rollout Generation"): of N proxy rewards per prompt keep the K/2
highest and the K/2 lowest candidates (N = 96, K = 24 in the paper) and preserve their initial
noise seeds.  Eq. (GRPO advantage, Section 2): A_i = (R_i - mu_R) / sigma_R with the population
standard deviation.  Appendix ("Group-Relative Ranking Consistency"): Kendall's tau, Spearman's
rho and the Top/Bottom-k match between two reward vectors.

Readings where the paper is silent:
  * ties: among equal rewards the lower candidate index ranks higher (rank 0 = highest reward);
  * output order: the K/2 best in descending order of reward, then the K/2 worst starting from
    the lowest;
  * Kendall's tau is tau-a, (concordant - discordant) / (N (N-1) / 2), a tied pair counting 0;
  * Spearman's rho is computed from the ordinal ranks above, 1 - 6 sum d^2 / (N (N^2 - 1));
  * Top/Bottom-k match = |top_k(ref) & top_k(proxy)| / k (and the same for the k lowest);
  * sigma_R = 0 (all rewards equal): advantages are 0.
Everything integer is exact; the advantages are FP64.
"""
from __future__ import annotations

import numpy as np


def descending_ranks(r: np.ndarray) -> np.ndarray:
    """rank[i] = number of candidates that beat i (higher reward, or equal reward and lower index)."""
    r = np.asarray(r, dtype=np.float64)
    n = r.shape[0]
    order = sorted(range(n), key=lambda i: (-r[i], i))   # a library sort as one step
    ranks = np.empty(n, np.int64)
    for pos, i in enumerate(order):
        ranks[i] = pos
    return ranks


def select_contrastive(rewards: np.ndarray, K: int) -> np.ndarray:
    """[P, N] rewards -> [P, K] candidate indices: K/2 best (descending), then K/2 worst (from the lowest)."""
    rewards = np.asarray(rewards, dtype=np.float64)
    P, N = rewards.shape
    if K % 2 or K > N or K <= 0:
        raise ValueError("K must be even and 0 < K <= N")
    out = np.empty((P, K), np.int32)
    for p in range(P):
        ranks = descending_ranks(rewards[p])
        by_rank = np.empty(N, np.int64)
        by_rank[ranks] = np.arange(N)
        out[p, : K // 2] = by_rank[: K // 2]
        out[p, K // 2:] = by_rank[::-1][: K // 2]
    return out


def group_advantages(rewards: np.ndarray) -> np.ndarray:
    """A = (R - mean) / population std per prompt, FP64; zeros where the std is 0."""
    rewards = np.asarray(rewards, dtype=np.float64)
    mu = rewards.mean(axis=1, keepdims=True)
    var = ((rewards - mu) ** 2).mean(axis=1, keepdims=True)
    sd = np.sqrt(var)
    return np.where(sd > 0, (rewards - mu) / np.where(sd > 0, sd, 1.0), 0.0)


def rank_consistency(ref: np.ndarray, proxy: np.ndarray, k: int):
    """Per prompt: (concordant - discordant pairs, sum of squared rank differences, top-k matches,
    bottom-k matches) as integers, and (tau, rho, top match rate, bottom match rate) as FP64."""
    ref, proxy = np.asarray(ref, dtype=np.float64), np.asarray(proxy, dtype=np.float64)
    P, N = ref.shape
    ints = np.zeros((P, 4), np.int64)
    for p in range(P):
        s = 0
        for i in range(N):
            for j in range(i + 1, N):
                s += int(np.sign(ref[p, i] - ref[p, j]) * np.sign(proxy[p, i] - proxy[p, j]))
        ra, rb = descending_ranks(ref[p]), descending_ranks(proxy[p])
        ints[p] = (s, int(((ra - rb) ** 2).sum()), int(((ra < k) & (rb < k)).sum()),
                   int(((ra >= N - k) & (rb >= N - k)).sum()))
    pairs = N * (N - 1) / 2
    floats = np.stack([ints[:, 0] / pairs, 1.0 - 6.0 * ints[:, 1] / (N * (N * N - 1.0)), ints[:, 2] / k,
                       ints[:, 3] / k], axis=1)
    return ints, floats
