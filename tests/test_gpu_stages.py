"""Bit-exact parity of the integer stages against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import sparsepr_oracle as orc
from paper_2608_18484_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,C,r", [(5000, 100, 48), (3001, 37, 64), (777, 300, 20), (64, 1, 7), (130, 130, 16), (6000, 1100, 64)])
def test_assign_bit_exact(n, C, r):
    rng = np.random.default_rng(n + C)
    X = rng.normal(size=(n, r)).astype(np.float32)
    mu = X[rng.choice(n, C, replace=False)] + rng.normal(size=(C, r)).astype(np.float32) * 0.3
    a = B.sparsepr_stage_assign(torch.from_numpy(X).cuda(), torch.from_numpy(mu).cuda()).cpu().numpy()
    assert np.array_equal(a, orc.kmeans_assign(X, mu))


def test_assign_ties_and_near_ties():
    rng = np.random.default_rng(1)
    n, C, r = 4000, 64, 48
    X = rng.normal(size=(n, r)).astype(np.float32)
    mu = rng.normal(size=(C, r)).astype(np.float32)
    mu[40] = mu[3]                                           # exact duplicate: tie -> lowest id
    mu[41] = mu[5] * np.float32(1 + 2e-7)                    # near duplicate: decided by the exact recheck
    X[:C] = mu                                               # rows sitting on centroids
    X[100:200] = ((mu[7].astype(np.float64) + mu[9]) / 2).astype(np.float32)   # equidistant up to rounding
    a = B.sparsepr_stage_assign(torch.from_numpy(X).cuda(), torch.from_numpy(mu).cuda()).cpu().numpy()
    ref = orc.kmeans_assign(X, mu)
    assert np.array_equal(a, ref)
    assert not np.any(a == 40)


def test_assign_large_magnitudes():
    rng = np.random.default_rng(2)
    X = (rng.normal(size=(3000, 64)) * 50 + 200).astype(np.float32)     # large common offset: cancellation-prone
    mu = X[:200].copy()
    a = B.sparsepr_stage_assign(torch.from_numpy(X).cuda(), torch.from_numpy(mu).cuda()).cpu().numpy()
    assert np.array_equal(a, orc.kmeans_assign(X, mu))


@pytest.mark.parametrize("n,C", [(100000, 591), (4096, 64), (33, 40), (1, 1), (75600, 2048)])
def test_permute_bit_exact(n, C):
    rng = np.random.default_rng(n)
    a = rng.integers(0, C, size=n).astype(np.int32)
    a[a == C // 2] = 0                                       # an empty group
    perm, inv, off = [t.cpu().numpy() for t in B.sparsepr_stage_permute(torch.from_numpy(a).cuda(), C)]
    p0, i0, o0 = orc.group_permutation(a, C)
    assert np.array_equal(perm, p0) and np.array_equal(inv, i0) and np.array_equal(off, o0)


def _route_case(rng, Cq, Ck, ties):
    n_q = rng.integers(0, 300, size=Cq).astype(np.int32)
    n_k = rng.integers(0, 300, size=Ck).astype(np.int32)
    score = rng.random((Cq, Ck)).astype(np.float32) ** 4
    if ties:
        score = np.round(score * 8) / 8
    return score.astype(np.float32), n_q, n_k


@pytest.mark.parametrize("Cq,Ck,ties", [(64, 64, False), (256, 256, False), (591, 591, False), (50, 70, True),
                                        (7, 1, True), (1, 9, False)])
def test_route_bit_exact(Cq, Ck, ties):
    rng = np.random.default_rng(Cq * 1000 + Ck)
    score, n_q, n_k = _route_case(rng, Cq, Ck, ties)
    total = int(n_q.astype(np.int64).sum() * n_k.astype(np.int64).sum())
    for frac in (0.0, 0.1, 0.25, 0.6, 1.0):
        budget = int(frac * total)
        ptr, idx, pairs = B.sparsepr_stage_route(torch.from_numpy(score).cuda(), torch.from_numpy(n_q).cuda(),
                                                 torch.from_numpy(n_k).cuda(), budget)
        p0, i0, pr0 = orc.route_select(score, n_q, n_k, budget)
        ptr, idx = ptr.cpu().numpy(), idx.cpu().numpy()
        assert np.array_equal(ptr, p0)
        assert np.array_equal(idx[:ptr[-1]], i0)
        assert int(pairs.item()) == pr0
    ptr, idx, pairs = B.sparsepr_stage_route(torch.from_numpy(score).cuda(), torch.from_numpy(n_q).cuda(),
                                             torch.from_numpy(n_k).cuda(), 0, select_all=True)
    p0, i0, pr0 = orc.route_select(score, n_q, n_k, 0, select_all=True)
    assert np.array_equal(ptr.cpu().numpy(), p0) and np.array_equal(idx.cpu().numpy()[:p0[-1]], i0)
    assert int(pairs.item()) == pr0 == total


def test_route_all_scores_equal():
    """Degenerate input: every cell ties, the selection is the (a,b)-ordered prefix."""
    score = np.full((20, 30), 0.5, np.float32)
    n_q = np.full(20, 10, np.int32)
    n_k = np.arange(1, 31).astype(np.int32)
    for budget in (0, 5000, 40000, 10**7):
        ptr, idx, pairs = B.sparsepr_stage_route(torch.from_numpy(score).cuda(), torch.from_numpy(n_q).cuda(),
                                                 torch.from_numpy(n_k).cuda(), budget)
        p0, i0, pr0 = orc.route_select(score, n_q, n_k, budget)
        assert np.array_equal(ptr.cpu().numpy(), p0) and np.array_equal(idx.cpu().numpy()[:p0[-1]], i0)
        assert int(pairs.item()) == pr0
