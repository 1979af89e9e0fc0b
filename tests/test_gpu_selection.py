"""GPU parity: stage-1 selection, advantages and rank-consistency metrics against the oracle."""
import numpy as np
import pytest
import torch

from oracle import selection as S

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2604_06916_b200 import binding
    binding.lib()
    return binding


def rewards(P, N, seed, ties=False):
    g = torch.Generator(device="cuda").manual_seed(seed)
    r = torch.randn(P, N, generator=g, device="cuda") * 0.8 + 0.3
    if ties:
        r = torch.round(r * 4) / 4      # many equal rewards: the tie rule decides
    return r.contiguous()


@pytest.mark.parametrize("P,N,K,ties", [(48, 96, 24, False), (48, 96, 24, True), (3, 2, 2, False), (5, 97, 96, True),
                                        (2, 4096, 64, False), (300, 7, 6, True)])
def test_selection_indices_seeds_and_advantages(B, P, N, K, ties):
    r = rewards(P, N, P + N + K, ties)
    seeds = torch.randint(0, 2 ** 62, (P, N), device="cuda", dtype=torch.int64,
                          generator=torch.Generator(device="cuda").manual_seed(9))
    idx, sel, adv = B.solrl_select_contrastive(r, K, seeds)
    torch.cuda.synchronize()
    rn = r.cpu().numpy()
    want = S.select_contrastive(rn, K)
    assert np.array_equal(idx.cpu().numpy(), want)
    assert np.array_equal(sel.cpu().numpy(), np.take_along_axis(seeds.cpu().numpy(), want.astype(np.int64), axis=1))
    A = S.group_advantages(rn)
    assert np.max(np.abs(adv.cpu().numpy() - A)) <= 2.0 ** -22 * max(1.0, np.abs(A).max())


def test_constant_rewards_give_zero_advantages_and_index_order(B):
    r = torch.full((2, 10), 1.5, device="cuda")
    idx, _, adv = B.solrl_select_contrastive(r, 4)
    assert idx.cpu().tolist() == [[0, 1, 9, 8]] * 2
    assert torch.count_nonzero(adv).item() == 0


@pytest.mark.parametrize("P,N,k,ties", [(48, 96, 4, False), (48, 96, 12, True), (4, 2, 1, False), (3, 2048, 16, False),
                                        (100, 33, 33, True)])
def test_rank_consistency_counts_exact(B, P, N, k, ties):
    ref = rewards(P, N, 11 * P + N, ties)
    g = torch.Generator(device="cuda").manual_seed(5)
    proxy = (ref + 0.25 * torch.randn(P, N, generator=g, device="cuda")).contiguous()
    if ties:
        proxy = torch.round(proxy * 4) / 4
    counts, metrics = B.solrl_rank_consistency(ref, proxy, k)
    torch.cuda.synchronize()
    ints, fl = S.rank_consistency(ref.cpu().numpy(), proxy.cpu().numpy(), k)
    assert np.array_equal(counts.cpu().numpy(), ints)
    assert np.max(np.abs(metrics.cpu().numpy() - fl)) <= 2.0 ** -23


def test_rejects_bad_arguments(B):
    r = torch.zeros((2, 8), device="cuda")
    with pytest.raises(B.SolError):
        B.solrl_select_contrastive(r, 5)        # K must be even
    with pytest.raises(B.SolError):
        B.solrl_select_contrastive(r, 10)       # K > N
    with pytest.raises(B.SolError):
        B.solrl_rank_consistency(r, r, 9)       # k > N
