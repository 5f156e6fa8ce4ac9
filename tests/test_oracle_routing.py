"""Pins for the oracle's router and probe selection (Section 4.3, Algorithm A.1)."""
import itertools
import os

import numpy as np

from oracle import sparsepr_oracle as orc


def _cells(ptr, idx):
    return {(a, int(b)) for a in range(len(ptr) - 1) for b in idx[ptr[a]:ptr[a + 1]]}


def _random_problem(rng, Cq, Ck, empty=True):
    n_q = rng.integers(1, 40, size=Cq)
    n_k = rng.integers(1, 40, size=Ck)
    if empty:
        n_q[rng.integers(0, Cq)] = 0
        n_k[rng.integers(0, Ck)] = 0
    score = rng.random((Cq, Ck)).astype(np.float32)
    return score, n_q, n_k


def test_cell_scores_definition():
    rng = np.random.default_rng(0)
    theta, kappa = rng.normal(size=(4, 5)), rng.normal(size=(6, 5))
    n_q, n_k = np.array([3, 0, 2, 9]), np.array([4, 1, 0, 7, 2, 5])
    p = orc.cell_scores(theta, kappa, n_q, n_k, 0.6)
    assert p.dtype == np.float32
    for a in range(4):
        e = np.exp(0.6 * kappa @ theta[a])
        ref = e / (n_k * e).sum()
        ref[n_k == 0] = 0
        if n_q[a] == 0:
            ref[:] = 0
        assert np.allclose(p[a], ref, rtol=1e-6)
        if n_q[a]:
            assert abs((p[a].astype(np.float64) * n_k).sum() - 1) < 1e-6     # weights over all keys sum to 1


def test_pair_budget():
    assert orc.pair_budget(0.25, 4096, 4096, 32) == 4096 * 4096 // 4 - 32 * 4096
    assert orc.pair_budget(0.001, 100, 100, 50) == 0
    # the float32 value of the density is what counts
    assert orc.pair_budget(0.22, 75600, 75600, 128) == int(np.floor(float(np.float32(0.22)) * 75600.0 * 75600.0)) - 128 * 75600


def test_route_invariants():
    rng = np.random.default_rng(1)
    for trial in range(20):
        Cq, Ck = rng.integers(2, 9), rng.integers(2, 9)
        score, n_q, n_k = _random_problem(rng, Cq, Ck)
        total = int(n_q.sum() * n_k.sum())
        prev = None
        for frac in (0.0, 0.2, 0.5, 0.8):
            budget = int(frac * total)
            ptr, idx, pairs = orc.route_select(score, n_q, n_k, budget)
            cells = _cells(ptr, idx)
            assert pairs == sum(int(n_q[a] * n_k[b]) for a, b in cells)
            assert pairs == orc.routed_pairs(n_q, n_k, ptr, idx)
            for a in range(Cq):
                row = idx[ptr[a]:ptr[a + 1]]
                assert np.all(np.diff(row) > 0)                       # ascending inside a row
                assert (len(row) > 0) == (n_q[a] > 0)                 # no non-empty group without support
                assert all(n_k[b] > 0 for b in row)
                if n_q[a]:
                    live = np.where(n_k > 0, score[a], -1)
                    assert int(np.argmax(live)) in row                # its best cell is always kept
            forced = sum(int(n_q[a] * n_k[int(np.argmax(np.where(n_k > 0, score[a], -1)))])
                         for a in range(Cq) if n_q[a])
            assert pairs <= max(budget, forced)
            # maximal prefix: the best unselected cell would not fit
            rest = [(float(score[a, b]), a, b) for a in range(Cq) for b in range(Ck)
                    if n_q[a] and n_k[b] and (a, b) not in cells]
            if rest:
                s, a, b = sorted(rest, key=lambda t: (-t[0], t[1], t[2]))[0]
                assert pairs + int(n_q[a] * n_k[b]) > budget
            if prev is not None:
                assert prev <= cells                                   # monotone in the budget
            prev = cells
        ptr, idx, pairs = orc.route_select(score, n_q, n_k, 0, select_all=True)
        assert pairs == total and _cells(ptr, idx) == {(a, b) for a in range(Cq) for b in range(Ck) if n_q[a] and n_k[b]}


def test_route_brute_force_prefix():
    """Tiny case, all steps by hand: 2x3 cells, unit-free sizes."""
    score = np.array([[0.5, 0.9, 0.1], [0.3, 0.2, 0.8]], dtype=np.float32)
    n_q, n_k = np.array([2, 3]), np.array([1, 2, 4])
    # forced: (0,1) cost 4, (1,2) cost 12 -> 16.  Rest by score: (0,0)=.5 cost 2, (1,0)=.3 cost 3,
    # (1,1)=.2 cost 6, (0,2)=.1 cost 8.
    expect = {16: {(0, 1), (1, 2)}, 17: {(0, 1), (1, 2)}, 18: {(0, 1), (1, 2), (0, 0)},
              21: {(0, 1), (1, 2), (0, 0), (1, 0)}, 26: {(0, 1), (1, 2), (0, 0), (1, 0)},
              27: {(0, 1), (1, 2), (0, 0), (1, 0), (1, 1)}, 3: {(0, 1), (1, 2)}}
    for budget, cells in expect.items():
        ptr, idx, pairs = orc.route_select(score, n_q, n_k, budget)
        assert _cells(ptr, idx) == cells
    # equal scores: order by (a, b)
    score[:] = 0.5
    ptr, idx, _ = orc.route_select(score, n_q, n_k, 2 + 8 + 2)     # forced (0,0)=2,(1,0)=3; then (0,1)=4 fits, (0,2)=8 does not
    assert _cells(ptr, idx) == {(0, 0), (1, 0), (0, 1)}


def test_probe_selection_toy_hand_execution():
    path = os.path.join(os.path.dirname(__file__), "golden", "probe_selection_toy.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    a = np.array([int(r[1]) for r in rows])
    phi = np.array([[float(r[2])] for r in rows])
    probes, w = orc.probe_select(a, phi, 3, 5)
    assert list(probes) == [3, 1, 2, 0, 5]
    assert np.allclose(w, [1.5, 1, 1, 1.5, 1])
    probes, w = orc.probe_select(a, phi, 3, 2)                     # M smaller than the group count
    assert list(probes) == [3, 1] and np.allclose(w, [3, 1])
    probes, w = orc.probe_select(a, phi, 3, 99)                    # M >= N_q: every row
    assert sorted(probes) == list(range(6)) and np.allclose(w, 1)


def test_probe_weights_cover_groups():
    rng = np.random.default_rng(2)
    a = rng.integers(0, 12, size=300)
    a[a == 7] = 8
    phi = rng.normal(size=(300, 5))
    for M in (5, 11, 40, 299):
        probes, w = orc.probe_select(a, phi, 12, M)
        assert len(set(probes.tolist())) == M
        sizes = np.bincount(a, minlength=12)
        m_a = np.bincount(a[probes], minlength=12)
        for g in range(12):
            if m_a[g]:
                assert abs(w[a[probes] == g].sum() - sizes[g]) < 1e-12   # sum of weights in a group = |G_a|
        # round-robin: probe counts differ by at most one among groups that still had rows
        assert all(m_a[g] >= min(sizes[g], m_a.max() - 1) for g in range(12))
        # inside a group the chosen rows are the closest to the centroid
        for g in np.nonzero(m_a)[0]:
            mem = np.nonzero(a == g)[0]
            dist = np.linalg.norm(phi[mem] - phi[mem].mean(0), axis=1)
            chosen = set(probes[a[probes] == g].tolist())
            assert chosen == set(mem[np.argsort(dist, kind="stable")[:m_a[g]]].tolist())
