"""The workspace-free assignment entry point, for users of the library that cannot
allocate device memory themselves (their process has given all of it to a memory pool,
or they run where cudaMalloc's device-wide synchronisation is not allowed).

It must give exactly the assignments of sparsepr_stage_assign, which in turn are the
float64 decisions of the definition (checked here against the CPU oracle as well).  Two calls in a row with
different shapes check that data left in the shared scratch array by the first call does
not leak into the second.  This file sorts last so that a run stopping at the first
failure has already executed every other test."""
import numpy as np
import pytest
import torch

from oracle import sparsepr_oracle as orc
from paper_2608_18484_b200 import binding as B

pytestmark = pytest.mark.gpu


def _case(seed, n, C, r):
    rng = np.random.default_rng(seed)
    X = rng.normal(size=(n, r)).astype(np.float32)
    mu = X[rng.choice(n, C, replace=False)] + rng.normal(size=(C, r)).astype(np.float32) * 0.25
    mu[C // 2] = mu[0]                                   # a duplicate centroid: tie -> lowest id
    return torch.from_numpy(X).cuda(), torch.from_numpy(mu).cuda()


def test_static_assign_matches_workspace_assign_twice():
    # first call fills the scratch with a large, wide problem; the second is smaller and narrower
    for seed, (n, C, r) in enumerate([(16384, 1024, 64), (5000, 37, 20)]):
        X, mu = _case(seed, n, C, r)
        expect = B.sparsepr_stage_assign(X, mu)
        out = torch.full((n,), -1, dtype=torch.int32, device="cuda")     # allocated by the caller, as the contract says
        got = B.sparsepr_stage_assign_static(X, mu, out)
        torch.cuda.synchronize()
        assert torch.equal(got, expect)
        assert int(got.min()) >= 0 and int(got.max()) < C
        # the definition itself: argmin of the float64 squared distance, ties to the lowest id
        rows = np.random.default_rng(seed).choice(n, 2048, replace=False)
        want = orc.kmeans_assign(X.cpu().numpy()[rows], mu.cpu().numpy())
        assert np.array_equal(got.cpu().numpy()[rows], want)


def test_static_assign_rejects_oversized_problems():
    X, mu = _case(3, 64, 8, 16)
    out = torch.empty(64, dtype=torch.int32, device="cuda")
    L = B.lib()
    big = 16385
    assert L.sparsepr_stage_assign_static(big, 8, 16, X.data_ptr(), mu.data_ptr(), out.data_ptr(), None) == 2
    assert L.sparsepr_stage_assign_static(64, 1025, 16, X.data_ptr(), mu.data_ptr(), out.data_ptr(), None) == 2
    assert L.sparsepr_stage_assign_static(64, 8, 65, X.data_ptr(), mu.data_ptr(), out.data_ptr(), None) == 2
    assert L.sparsepr_stage_assign_static(0, 8, 16, X.data_ptr(), mu.data_ptr(), out.data_ptr(), None) == 1
    assert "unsupported" in B.status_string(2)
