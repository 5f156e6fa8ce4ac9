"""Pins for Response-Coupled Partitioning in the oracle (Section 4.1, Appendix B)."""
import numpy as np
import pytest

from oracle import sparsepr_oracle as orc


def test_splitmix64_known_sequence():
    # First outputs of the public-domain splitmix64 generator seeded with 0
    # (state advanced by the golden-ratio increment before every output).
    inc = 0x9E3779B97F4A7C15
    assert orc.splitmix64(0) == 0xE220A8397B1DCDAF
    assert orc.splitmix64(inc) == 0x6E789E6AA1B965F4
    assert orc.splitmix64((2 * inc) & (2**64 - 1)) == 0x06C45D188009454F


def test_stride_sample_properties():
    for n, N in [(64, 4096), (256, 32760), (591, 75600), (7, 7), (1, 5)]:
        for tag in (1, 2, 3):
            idx = orc.stride_sample(n, N, seed=0, tag=tag, bh=3)
            assert idx.min() >= 0 and idx.max() < N
            assert np.all(np.diff(idx) >= 1)                      # distinct, ascending
            assert np.all(np.abs(np.diff(idx) - N / n) <= 1.0)    # evenly spread
    a = orc.stride_sample(64, 4096, 0, 1, 0)
    assert not np.array_equal(a, orc.stride_sample(64, 4096, 0, 1, 1))   # offset depends on the head
    with pytest.raises(ValueError):
        orc.stride_sample(5, 4, 0, 1, 0)


def test_key_metric_identity():
    """(k_j-k_l)^T M_K (k_j-k_l) = ||Q_s (k_j-k_l)||^2 / M_s, and with r_K = d the
    feature distance equals it up to the unit-mean normalisation (Section 4.1)."""
    rng = np.random.default_rng(0)
    Qs, K = rng.normal(size=(20, 6)), rng.normal(size=(9, 6))
    M_K = orc.key_response_metric(Qs)
    F, lam = orc.eig_feature_map(M_K, 6)
    phi = orc.key_response(K, F)
    for j in range(9):
        for l in range(9):
            dk = K[j] - K[l]
            rhs = np.sum((Qs @ dk) ** 2) / 20
            assert abs(dk @ M_K @ dk - rhs) < 1e-12
            assert abs(np.sum((phi[j] - phi[l]) ** 2) * lam.mean() - rhs) < 1e-11


def test_feature_map_properties():
    rng = np.random.default_rng(1)
    A = rng.normal(size=(30, 8))
    Mm = A.T @ A / 30
    for r in (3, 8, 12):
        F, lam = orc.eig_feature_map(Mm, r)
        rr = min(r, 8)
        assert F.shape == (8, rr)
        assert abs(np.trace(F.T @ F) - rr) < 1e-12                # normalised eigenvalues have unit mean
        G = F.T @ F
        assert np.allclose(G, np.diag(np.diag(G)), atol=1e-12)    # columns are orthogonal eigendirections
        assert np.all(np.diff(np.diag(G)) <= 1e-12)               # leading first
        # columns are eigenvectors: M f = lambda f
        assert np.allclose(Mm @ F, F * lam[None, :], atol=1e-12)
        # F F^T is the rank-r truncation of M divided by the mean retained eigenvalue
        w, U = np.linalg.eigh(Mm)
        trunc = (U[:, -rr:] * w[-rr:]) @ U[:, -rr:].T
        assert np.allclose(F @ F.T * lam.mean(), trunc, atol=1e-12)
    F, _ = orc.eig_feature_map(np.zeros((4, 4)), 2)
    assert np.all(F == 0)


def test_query_metric_uniform_weighting():
    rng = np.random.default_rng(2)
    K = rng.normal(size=(40, 5))
    a = rng.integers(0, 6, size=40)
    a[a == 4] = 3                                                 # group 4 empty
    kappa, n = orc.kv_centroids(K, a, 6)
    assert n[4] == 0 and np.all(kappa[4] == 0)
    for b in range(6):
        if n[b]:
            assert np.allclose(kappa[b], K[a == b].mean(0), atol=1e-14)
    M_Q = orc.query_response_metric(kappa, n)
    rows = np.stack([K[a == b].mean(0) for b in range(6) if n[b]])
    rows = rows - rows.mean(0)
    assert np.allclose(M_Q, rows.T @ rows / (5 * 5), atol=1e-14)  # C_k^+ = 5 non-empty groups, d = 5
    # duplicating the tokens of one group changes nothing (equal weight per group)
    K2, a2 = np.concatenate([K, K[a == 2]]), np.concatenate([a, a[a == 2]])
    k2, n2 = orc.kv_centroids(K2, a2, 6)
    assert np.allclose(orc.query_response_metric(k2, n2), M_Q, atol=1e-14)


def test_query_response_normalisation():
    rng = np.random.default_rng(3)
    Q, F = rng.normal(size=(12, 7)), rng.normal(size=(7, 4))
    phi = orc.query_response(Q, F)
    assert np.allclose((phi ** 2).sum(1), 4.0, atol=1e-12)         # ||phi||^2 = r_Q
    assert np.allclose(orc.query_response(3.7 * Q, F), phi, atol=1e-12)   # positive scale invariance
    Y = Q @ F
    assert np.allclose(phi, Y / np.sqrt((Y ** 2).mean(1, keepdims=True)), atol=1e-12)
    Q0 = Q.copy(); Q0[5] = 0
    assert np.all(orc.query_response(Q0, F)[5] == 0)               # clamp: zero row stays zero
    tiny = orc.query_response(1e-9 * Q[:1], F, eps=1e-6)
    assert np.allclose(tiny, 1e-9 * Y[:1] / 1e-6)                  # below eps the divisor is eps


def test_kmeans_assign_brute_force_and_ties():
    rng = np.random.default_rng(4)
    X, mu = rng.normal(size=(50, 5)), rng.normal(size=(7, 5))
    a = orc.kmeans_assign(X, mu, chunk=16)
    for j in range(50):
        dist = [sum((X[j, k] - mu[c, k]) ** 2 for k in range(5)) for c in range(7)]
        assert a[j] == dist.index(min(dist))
    mu2 = np.concatenate([mu[3:4], mu])                            # duplicate centroid 3 at id 0
    a2 = orc.kmeans_assign(X, mu2)
    assert np.all(a2[a == 3] == 0) and np.all(a2[a != 3] == a[a != 3] + 1)   # ties go to the lowest id


def test_kmeans_invariants():
    rng = np.random.default_rng(5)
    centers = rng.normal(size=(6, 4)) * 20
    lab = np.repeat(np.arange(6), 30)
    X = centers[lab] + rng.normal(size=(180, 4))
    init = np.arange(6) * 30                                       # one point of each planted cluster
    a, mu = orc.kmeans(X, 6, init, T=5)
    assert np.array_equal(a, lab)                                   # planted clusters recovered
    # objective is non-increasing over iterations
    prev = np.inf
    for T in range(1, 6):
        aT, muT = orc.kmeans(X + rng.normal(size=X.shape) * 0, 6, [0, 1, 2, 3, 4, 5], T)
        obj = orc.kmeans_objective(X, muT, aT)
        assert obj <= prev + 1e-9
        prev = obj
    a1, _ = orc.kmeans(X, 1, [17], T=3)
    assert np.all(a1 == 0)
    aN, _ = orc.kmeans(X, 180, np.arange(180), T=3)
    assert np.array_equal(aN, np.arange(180))                       # C = N: every point its own cluster
    # an empty cluster keeps its centroid: two identical start rows
    Xd = np.concatenate([X, X[:1]])
    a1st, _ = orc.kmeans(Xd, 2, [0, 180], T=1)
    assert np.all(a1st == 0)                                        # duplicate centroids: tie to id 0
    _, mud = orc.kmeans(Xd, 2, [0, 180], T=2)
    assert np.allclose(mud[0], Xd.mean(0)) and np.array_equal(mud[1], X[0])   # empty cluster 1 kept its centroid


def test_kmeans_matches_sklearn_lloyd():
    sk = pytest.importorskip("sklearn.cluster")
    rng = np.random.default_rng(6)
    X = rng.normal(size=(300, 6))
    init = orc.stride_sample(10, 300, 0, 2, 0)
    km = sk.KMeans(n_clusters=10, init=X[init], n_init=1, algorithm="lloyd", max_iter=4, tol=0.0).fit(X)
    # sklearn's max_iter=4 runs 4 (assign, update) rounds and then labels the
    # points against the last centroids: 5 assignments in this oracle's count
    a, mu = orc.kmeans(X, 10, init, T=5)
    assert np.array_equal(a, km.labels_)
    assert np.allclose(mu, km.cluster_centers_, atol=1e-10)


def test_kmeans_warm_start():
    """Warm start from a previous partition: the seeds are the group means of the current features (checked
    against sklearn's Lloyd started from independently computed means), a cluster the previous partition left
    empty starts from its strided row, and a planted partition is a fixed point that one pass reproduces."""
    sk = pytest.importorskip("sklearn.cluster")
    rng = np.random.default_rng(16)
    X = rng.normal(size=(400, 5))
    init = orc.stride_sample(8, 400, 0, 2, 0)
    prev = rng.integers(0, 8, size=400)
    prev[prev == 3] = 4                                           # cluster 3 empty in the previous partition
    seeds = np.stack([X[prev == c].mean(0) if (prev == c).any() else X[init[c]] for c in range(8)])
    km = sk.KMeans(n_clusters=8, init=seeds, n_init=1, algorithm="lloyd", max_iter=3, tol=0.0).fit(X)
    a, mu = orc.kmeans(X, 8, init, T=4, init_assign=prev)
    assert np.array_equal(a, km.labels_) and np.allclose(mu, km.cluster_centers_, atol=1e-10)
    a1, mu1 = orc.kmeans(X, 8, init, T=1, init_assign=prev)
    assert np.array_equal(a1, orc.kmeans_assign(X, seeds)) and np.allclose(mu1, seeds)
    # well separated planted clusters: the planted partition reproduces itself in one pass, whatever the strided rows are
    centers = rng.normal(size=(6, 4)) * 20.0
    lab = rng.integers(0, 6, size=300)
    Y = centers[lab] + rng.normal(size=(300, 4)) * 0.1
    a2, _ = orc.kmeans(Y, 6, orc.stride_sample(6, 300, 0, 3, 1), T=1, init_assign=lab)
    assert np.array_equal(a2, lab)
    # the objective does not rise along a warm-started run either
    objs = []
    for T in range(1, 6):
        aT, muT = orc.kmeans(X, 8, init, T=T, init_assign=prev)
        objs.append(orc.kmeans_objective(X, muT, aT))
    assert all(objs[i + 1] <= objs[i] + 1e-9 for i in range(len(objs) - 1))


def test_partition_variants():
    """Semantic reference partition = Lloyd on the raw activations (checked against sklearn from the same rows);
    the key-response K/V variant takes its K/V groups from the method and its query groups from the semantic
    partition; every variant yields a complete, valid plan."""
    sk = pytest.importorskip("sklearn.cluster")
    rng = np.random.default_rng(21)
    N, d, C = 384, 16, 6
    cent = rng.normal(size=(C, d)) * 2.0
    lab = rng.integers(0, C, size=N)
    Q = cent[lab] + rng.normal(size=(N, d)) * 0.5
    K = 0.7 * cent[lab] + rng.normal(size=(N, d)) * 0.5
    prm = orc.default_params(density=0.4, block=64, n_sample=64, n_probe=8, rK=8, rQ=8, kmeans_iters=4, softmax_scale=1.0)
    plans = {v: orc.plan_head(Q, K, dict(prm, partition=v), 3) for v in (0, 1, 2)}
    for X, key, tag in ((K, "a_K", orc.TAG_KV_INIT), (Q, "a_Q", orc.TAG_Q_INIT)):
        init = orc.stride_sample(C, N, 0, tag, 3)
        km = sk.KMeans(n_clusters=C, init=X[init], n_init=1, algorithm="lloyd", max_iter=3, tol=0.0).fit(X)
        assert np.array_equal(plans[2][key], km.labels_)
    assert np.array_equal(plans[1]["a_K"], plans[0]["a_K"]) and np.array_equal(plans[1]["a_Q"], plans[2]["a_Q"])
    assert not np.array_equal(plans[0]["a_Q"], plans[2]["a_Q"])
    budget = orc.pair_budget(0.4, N, N, 8)
    for v, p in plans.items():
        assert p["routed_pairs"] <= budget and len(set(p["probe_idx"].tolist())) == 8
        assert np.all(np.diff(p["route_ptr"]) >= (p["n_q"] > 0))


def test_grouped_query_plan():
    """K/V side shared by the query heads of a group: with one query head it is the single-head plan; with several,
    the key-response metric is the second moment of all their sampled rows, the K/V partition is common, and each
    query head has its own query partition and routes against the shared K/V groups."""
    rng = np.random.default_rng(31)
    N, d = 320, 16
    K = rng.normal(size=(N, d))
    Qs = [rng.normal(size=(N, d)) + 0.5 * K for _ in range(3)]
    prm = orc.default_params(density=0.4, block=64, n_sample=32, n_probe=8, rK=8, rQ=8, kmeans_iters=3, softmax_scale=1.0)
    single = orc.plan_head(Qs[0], K, prm, 5)
    group1 = orc.plan_group(Qs[:1], K, prm, 5, 5)[0]
    for key in ("a_K", "a_Q", "route_idx", "probe_idx", "M_K", "F_Q"):
        assert np.array_equal(single[key], group1[key]), key
    plans = orc.plan_group(Qs, K, prm, 2, 6)
    rows = np.concatenate([Q[orc.stride_sample(32, N, 0, orc.TAG_QUERY_SAMPLE, 6 + g)] for g, Q in enumerate(Qs)])
    assert np.allclose(plans[0]["M_K"], rows.T @ rows / rows.shape[0], atol=1e-14)
    assert all(np.array_equal(p["a_K"], plans[0]["a_K"]) and p["kappa"] is plans[0]["kappa"] for p in plans)
    assert np.array_equal(plans[0]["a_K"], orc.kmeans(plans[0]["phi_K"], 5, orc.stride_sample(5, N, 0, orc.TAG_KV_INIT, 2), 3)[0])
    assert not np.array_equal(plans[0]["a_Q"], plans[1]["a_Q"])
    budget = orc.pair_budget(0.4, N, N, 8)
    for g, p in enumerate(plans):
        assert np.array_equal(p["a_Q"], orc.kmeans(p["phi_Q"], 5, orc.stride_sample(5, N, 0, orc.TAG_Q_INIT, 6 + g), 3)[0])
        assert p["routed_pairs"] <= budget
        assert p["routed_pairs"] == orc.routed_pairs(p["n_q"], p["n_k"], p["route_ptr"], p["route_idx"])


def test_group_permutation():
    rng = np.random.default_rng(7)
    a = rng.integers(0, 9, size=100)
    a[a == 5] = 6
    perm, inv, off = orc.group_permutation(a, 9)
    assert np.array_equal(inv[perm], np.arange(100)) and np.array_equal(perm[inv], np.arange(100))
    assert np.all(np.diff(a[perm]) >= 0)
    assert np.array_equal(np.diff(off), np.bincount(a, minlength=9)) and off[0] == 0 and off[-1] == 100
    for g in range(9):
        seg = perm[off[g]:off[g + 1]]
        assert np.all(a[seg] == g) and np.all(np.diff(seg) > 0)     # original order inside a group
