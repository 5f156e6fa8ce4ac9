"""Stage-by-stage parity of the GPU plan (stages 1-2 of the call) with the fp64 oracle.

The plan is a chain of discrete decisions (two k-means runs, the route cut, the probe
ranking) taken on floating-point quantities, so one flipped near-tie early in the chain
changes everything after it.  Each link is therefore checked on its own: the oracle is
fed what the GPU decided up to that link and evaluates the link itself in float64; the
GPU's continuous quantities are compared with a tolerance, its decisions must agree
except where the oracle's own quantities are within a stated margin of a tie.

    a1-a3  F_K F_K^T (gauge-free form of the key-response map; eigenvector signs are arbitrary)
    a4     a_K against k-means from scratch
    a5     kappa, and F_Q F_Q^T from the centroid metric of the GPU's own K/V groups
    a6     phi_Q: row norms and Gram entries on a row sample (invariant to the gauge of F_Q)
    a7     a_Q against k-means on the oracle's phi_Q (same initial rows)
    a9     theta, cell scores; selected cells against route_select on the oracle's scores
    a10    probe set, order and weights against Algorithm A.1 on the oracle's distances
"""
import numpy as np
import pytest

from oracle import sparsepr_oracle as orc
from paper_2608_18484_b200 import binding as B
from paper_2608_18484_b200 import workloads as W
from tests.gpu_util import heads_to_device

pytestmark = pytest.mark.gpu

CASES = [("tiny-f32", W.TINY), ("480p-like-bf16", W.VIDEO_480P.scaled(grid=(3, 30, 52), H=2, n_probe=64))]

# Tolerances.  float32 tensors run the eigen-solver and the fit in float64 on the GPU and the
# projections in float32; bf16 tensors run the eigen-solver in float32 and the projections on the
# tensor cores with a three-term bf16 split of F (2^-24 relative).  The continuous quantities are then
# accurate to a few float32 ulps times a condition number (eigen-gap for F F^T, exp for the scores).
TOL = {
    "f32": dict(FF=1e-5, kappa=2e-6, gram=1e-5, norm=1e-5, score=1e-4, agree_K=0.97, agree_Q=0.97, obj=2e-3),
    "bf16": dict(FF=1e-4, kappa=2e-6, gram=1e-4, norm=2e-5, score=1e-4, agree_K=0.97, agree_Q=0.97, obj=2e-3),
}
TIE = 5e-3          # relative margin inside which two oracle scores / distances count as tied


def rel_fro(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def plan_links(wl, i, Q, K, exp, feat, prm, warm=None, ref=None, kv=None):
    """Everything the assertions need for head i: GPU quantities beside the oracle's evaluation of each link.
    `warm` = the partition {"a_K", "a_Q"} that a warm-started GPU plan was seeded with.  Under grouped-query
    attention `kv` is the index of the head's K/V head (the K/V-side arrays have one entry per K/V head) and `ref`
    the oracle's plan of this query head inside its group."""
    N, d = Q.shape
    C = -(-N // wl.block)
    out = {}
    if ref is None:
        ref = orc.plan_head(Q, K, prm, i, warm=warm)
    kv = i if kv is None else kv
    variant = prm.get("partition", 0)
    aK, aQ = exp["kv_assign"][kv], exp["q_assign"][i]
    # a1-a3 (a semantic K/V partition clusters K itself: no feature map)
    out["FF_K"] = 0.0
    if variant != orc.PARTITION_SEMANTIC:
        FK = feat["F_K"][kv].astype(np.float64)
        out["FF_K"] = rel_fro(FK @ FK.T, ref["F_K"] @ ref["F_K"].T)
    # a4
    out["agree_K"] = float((aK == ref["a_K"]).mean())
    out["obj_K"] = orc.kmeans_objective(ref["phi_K"], _means(ref["phi_K"], aK, C), aK) / \
        orc.kmeans_objective(ref["phi_K"], _means(ref["phi_K"], ref["a_K"], C), ref["a_K"]) - 1.0
    # a5: centroids and query metric of the GPU's own K/V groups
    kappa, n_k = orc.kv_centroids(K, aK, C)
    out["kappa"] = float(np.abs(feat["kappa"][kv] - kappa).max())
    phi_gpu = feat["phi_Q"][i].astype(np.float64)
    rows = np.random.default_rng(5).choice(N, min(N, 384), replace=False)
    if variant == orc.PARTITION_RESPONSE_COUPLED:
        F_Q, _ = orc.eig_feature_map(orc.query_response_metric(kappa, n_k), prm["rQ"])
        FQ = feat["F_Q"][kv].astype(np.float64)
        out["FF_Q"] = rel_fro(FQ @ FQ.T, F_Q @ F_Q.T)
        # a6
        phi_ref = orc.query_response(Q, F_Q, prm["eps_rms"])
        out["norm"] = float(np.abs((phi_gpu ** 2).sum(axis=1) / phi_ref.shape[1] - 1.0).max())
    else:                                           # semantic query partition: the features are the queries themselves
        phi_ref = np.asarray(Q, dtype=np.float64)
        out["FF_Q"] = 0.0
        out["norm"] = float(np.abs(phi_gpu - phi_ref).max())
    out["gram"] = rel_fro(phi_gpu[rows] @ phi_gpu[rows].T, phi_ref[rows] @ phi_ref[rows].T)
    # a7
    aQ_ref, _ = orc.kmeans(phi_ref, C, orc.stride_sample(C, N, prm["seed"], orc.TAG_Q_INIT, i), prm["kmeans_iters"],
                           init_assign=None if warm is None else warm["a_Q"])
    out["agree_Q"] = float((aQ == aQ_ref).mean())
    out["obj_Q"] = orc.kmeans_objective(phi_ref, _means(phi_ref, aQ, C), aQ) / \
        orc.kmeans_objective(phi_ref, _means(phi_ref, aQ_ref, C), aQ_ref) - 1.0
    # a9: scores and selection on the GPU's own groups
    theta, n_q = orc.query_centroids(Q, aQ, C)
    out["theta"] = float(np.abs(feat["theta"][i] - theta).max())
    score = orc.cell_scores(theta, kappa, n_q, n_k, ref["scale"])
    g = feat["score"][i]
    live = score > 1e-30
    out["score"] = float(np.abs(g[live].astype(np.float64) / score[live] - 1.0).max())
    out["score_dead"] = float(np.abs(g[~live]).max()) if (~live).any() else 0.0
    budget = orc.pair_budget(prm["density"], N, N, ref["M"])
    rp, ri, pairs = orc.route_select(score, n_q, n_k, budget, select_all=np.float32(prm["density"]) >= 1.0)
    z_ref = np.zeros((C, C), bool)
    z_gpu = np.zeros((C, C), bool)
    ptr, idx = exp["route_ptr"][i], exp["route_idx"][i]
    for a in range(C):
        z_ref[a, ri[rp[a]:rp[a + 1]]] = True
        z_gpu[a, idx[ptr[a]:ptr[a + 1]]] = True
    diff = np.argwhere(z_ref != z_gpu)
    # the cut of the oracle's order: lowest score among its cells that are not a row's forced best cell
    forced = np.zeros((C, C), bool)
    rowbest = np.where(n_q > 0, np.argmax(np.where(n_k[None, :] > 0, score, -1.0), axis=1), -1)
    forced[np.nonzero(rowbest >= 0)[0], rowbest[rowbest >= 0]] = True
    free = z_ref & ~forced
    cut = float(score[free].min()) if free.any() else float("inf")
    out["route_cut"] = cut
    worst = 0.0
    for a, b in diff:
        s = float(score[a, b])
        near_cut = abs(s / cut - 1.0) if np.isfinite(cut) else float("inf")
        near_best = abs(s / float(score[a, rowbest[a]]) - 1.0)
        worst = max(worst, min(near_cut, near_best))
    out["route_diff_cells"] = int(len(diff))
    out["route_diff_margin"] = worst
    cost = n_q[:, None].astype(np.int64) * n_k[None, :].astype(np.int64)
    out["route_pairs_gap"] = abs(int(exp["routed_pairs"][i]) - pairs)
    out["route_diff_cost"] = int(cost[z_ref != z_gpu].sum())
    out["route_pairs_gpu"] = int(exp["routed_pairs"][i])
    out["budget"] = budget
    # a10: Algorithm A.1 on the GPU's groups with the oracle's distances
    M = ref["M"]
    P, w = exp["probe_idx"][i], exp["probe_w"][i]
    P_ref, w_ref = orc.probe_select(aQ, phi_ref, C, M)
    out["probe_groups_equal"] = bool(np.array_equal(aQ[P], aQ[P_ref]))            # same round-robin group sequence
    out["probe_w_equal"] = bool(np.array_equal(w, w_ref.astype(np.float32)))
    out["probe_distinct"] = len(set(P.tolist())) == M
    sizes = np.bincount(aQ, minlength=C)
    m_a = np.bincount(aQ[P], minlength=C)
    out["probe_m_equal"] = bool(np.array_equal(m_a, np.bincount(aQ[P_ref], minlength=C)))
    slack, order_ok = 0.0, True
    for a in np.nonzero(m_a)[0]:
        members = np.nonzero(aQ == a)[0]
        c_a = phi_ref[members].mean(axis=0)
        dist = np.sqrt(((phi_ref[members] - c_a) ** 2).sum(axis=1))
        kth = np.sort(dist)[m_a[a] - 1]
        mine = P[aQ[P] == a]                                                       # in selection order
        dm = np.sqrt(((phi_ref[mine] - c_a) ** 2).sum(axis=1))
        slack = max(slack, float((dm.max() - kth) / max(kth, 1e-12)))
        order_ok &= bool(np.all(np.diff(dm) >= -TIE * np.maximum(dm[:-1], 1e-12)))
    out["probe_slack"] = slack
    out["probe_order_ok"] = order_ok
    out["probe_same_set"] = float(len(set(P.tolist()) & set(P_ref.tolist())) / max(M, 1))
    out["sizes_max"] = int(sizes.max())
    return out


def _means(X, a, C):
    mu = np.zeros((C, X.shape[1]))
    np.add.at(mu, a, X)
    n = np.bincount(a, minlength=C)
    mu[n > 0] /= n[n > 0, None]
    return mu


def run_case(wl, **extra):
    heads = [0, 1]
    host, (Qd, Kd, Vd) = heads_to_device(wl, heads)
    kw = dict(density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
              softmax_scale=wl.softmax_scale, **extra)
    plan = B.sparsepr_plan(Qd, Kd, Vd, **kw)
    st = B.sparsepr_plan_stats(plan)
    exp = B.sparsepr_plan_export(plan)
    feat = B.sparsepr_plan_export_features(plan)
    prm = orc.default_params(**kw)
    return st, [plan_links(wl, i, Q, K, exp, feat, prm) for i, (Q, K, V) in enumerate(host)]


def check_links(wl, links):
    t = TOL[wl.dtype]
    for m in links:
        # continuous quantities
        assert m["FF_K"] <= t["FF"] and m["FF_Q"] <= t["FF"], m
        assert m["kappa"] <= t["kappa"] and m["theta"] <= t["kappa"], m
        assert m["gram"] <= t["gram"] and m["norm"] <= t["norm"], m
        assert m["score"] <= t["score"] and m["score_dead"] == 0.0, m
        # the two partitions: most rows agree, and the clustering the GPU found is as good as the oracle's
        assert m["agree_K"] >= t["agree_K"] and abs(m["obj_K"]) <= t["obj"], m
        assert m["agree_Q"] >= t["agree_Q"] and abs(m["obj_Q"]) <= t["obj"], m
        # routes: the same cells except cells tied (within TIE) with the cut or with a row's best cell
        assert m["route_diff_margin"] <= TIE, m
        assert m["route_pairs_gap"] <= m["route_diff_cost"] and m["route_pairs_gpu"] <= m["budget"], m
        # probes (Algorithm A.1, Appendix A.2): group sequence, counts and weights exactly; members up to ties
        assert m["probe_distinct"] and m["probe_groups_equal"] and m["probe_m_equal"] and m["probe_w_equal"], m
        assert m["probe_slack"] <= TIE and m["probe_order_ok"], m


@pytest.mark.parametrize("name,wl", CASES, ids=[c[0] for c in CASES])
def test_every_plan_link_matches_the_oracle(name, wl):
    st, links = run_case(wl)
    assert st["device_error"] == 0
    check_links(wl, links)


@pytest.mark.parametrize("name,wl", CASES, ids=[c[0] for c in CASES])
def test_warm_started_plan_matches_the_oracle(name, wl):
    """Two calls over the same scene (same centroid tables, fresh noise).  The second plan starts both k-means runs
    from the first plan's partition and runs 3 passes; the oracle, seeded with the GPU's first partition, must
    arrive at the same plan link by link.  Warm and cold plans must also differ (the seed is really used)."""
    heads = [0, 1]
    kw = dict(density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
              softmax_scale=wl.softmax_scale)
    _, (Q1, K1, V1) = heads_to_device(wl, heads)
    first = B.sparsepr_plan(Q1, K1, V1, **kw)
    e1 = B.sparsepr_plan_export(first)
    host2, (Q2, K2, V2) = heads_to_device(wl, heads, step=1)
    kw3 = dict(kw, kmeans_iters=3)
    second = B.sparsepr_plan(Q2, K2, V2, warm_from=first, **kw3)
    st = B.sparsepr_plan_stats(second)
    assert st["device_error"] == 0
    exp, feat = B.sparsepr_plan_export(second), B.sparsepr_plan_export_features(second)
    prm = orc.default_params(**kw3)
    links = [plan_links(wl, i, Q, K, exp, feat, prm, warm=dict(a_K=e1["kv_assign"][i], a_Q=e1["q_assign"][i]))
             for i, (Q, K, V) in enumerate(host2)]
    check_links(wl, links)
    cold = B.sparsepr_plan_export(B.sparsepr_plan(Q2, K2, V2, **kw3))
    assert not np.array_equal(cold["kv_assign"], exp["kv_assign"])
    # the warm plan drives a full call
    O = B.sparsepr_attend(second, Q2, K2, V2)
    assert bool(np.isfinite(O.float().cpu().numpy()).all())


@pytest.mark.parametrize("variant", [orc.PARTITION_KEY_RESPONSE_KV, orc.PARTITION_SEMANTIC], ids=["key-response-kv", "semantic"])
@pytest.mark.parametrize("name,wl", CASES, ids=[c[0] for c in CASES])
def test_partition_variants_match_the_oracle(name, wl, variant):
    """The ablation partitions (k-means on the raw activations for one or both sides; d = 64 on the tensor-core
    assignment, d = 128 on the CUDA-core one) link by link, and a full call on such a plan."""
    st, links = run_case(wl, partition=variant)
    assert st["device_error"] == 0
    check_links(wl, links)
    _, (Qd, Kd, Vd) = heads_to_device(wl, [0, 1])
    kw = dict(density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
              softmax_scale=wl.softmax_scale, partition=variant)
    plan = B.sparsepr_plan(Qd, Kd, Vd, **kw)
    O = B.sparsepr_attend(plan, Qd, Kd, Vd)
    assert bool(np.isfinite(O.float().cpu().numpy()).all()) and B.sparsepr_plan_stats(plan)["device_error"] == 0
