"""Grouped-query attention (Section 4.3): several query heads attend to one K/V head; the K/V partition and its
metadata are computed once per K/V head and shared, every query head keeps its own query partition, probes and
routes.  The GPU plan is checked link by link against the oracle's grouped plan, the outputs against the oracle's
evaluation of the GPU's plan, and the dense entry point against exact attention."""
import numpy as np
import pytest
import torch

from oracle import sparsepr_oracle as orc
from paper_2608_18484_b200 import binding as B
from paper_2608_18484_b200 import workloads as W
from tests.gpu_util import assert_bf16_close, to_np
from tests.test_gpu_plan_parity import check_links, plan_links

pytestmark = pytest.mark.gpu

G, HKV = 2, 2


def grouped_inputs(wl):
    """Hkv K/V heads; query head kv * G + g = the queries of K/V head kv's scene with a fresh noise draw g."""
    Ks, Vs, Qs = [], [], []
    for kv in range(HKV):
        Q0, K, V = W.make_head(wl, kv)
        Ks.append(K)
        Vs.append(V)
        Qs.append(Q0)
        for g in range(1, G):
            Qs.append(W.make_head(wl, kv, step=g)[0])
    dev = [torch.from_numpy(np.stack(x)[None]).to(torch.bfloat16).cuda().contiguous() for x in (Qs, Ks, Vs)]
    return Qs, Ks, Vs, dev


def test_grouped_query_call_matches_the_oracle():
    wl = W.VIDEO_480P.scaled(grid=(3, 30, 52), H=G * HKV, n_probe=64)
    Qs, Ks, Vs, (Qd, Kd, Vd) = grouped_inputs(wl)
    assert Qd.shape[1] == G * HKV and Kd.shape[1] == HKV
    kw = dict(density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
              softmax_scale=wl.softmax_scale)
    plan = B.sparsepr_plan(Qd, Kd, Vd, **kw)
    O, Osp = B.sparsepr_attend(plan, Qd, Kd, Vd, return_sparse=True)
    st = B.sparsepr_plan_stats(plan)
    assert st["device_error"] == 0
    exp, feat = B.sparsepr_plan_export(plan), B.sparsepr_plan_export_features(plan)
    assert exp["kv_assign"].shape[0] == HKV and exp["q_assign"].shape[0] == G * HKV
    prm = orc.default_params(**kw)
    links = []
    for kv in range(HKV):
        refs = orc.plan_group(Qs[kv * G:(kv + 1) * G], Ks[kv], prm, kv, kv * G)
        for g in range(G):
            i = kv * G + g
            links.append(plan_links(wl, i, Qs[i], Ks[kv], exp, feat, prm, ref=refs[g], kv=kv))
            # the outputs of this query head against the oracle's evaluation of the GPU's own plan
            ptr, idx = exp["route_ptr"][i], exp["route_idx"][i]
            gplan = dict(scale=wl.softmax_scale, M=wl.n_probe, a_Q=exp["q_assign"][i], a_K=exp["kv_assign"][kv],
                         route_ptr=ptr, route_idx=idx[:ptr[-1]], probe_idx=exp["probe_idx"][i],
                         probe_w=exp["probe_w"][i].astype(np.float64))
            O_hat, O_sp, _ = orc.attend_head(Qs[i], Ks[kv], Vs[kv], gplan, prm)
            assert_bf16_close(to_np(Osp[0, i]), O_sp)
            assert_bf16_close(to_np(O[0, i]), O_hat)
    check_links(wl, links)
    # the two query heads of a group share the K/V side and differ on the query side
    assert not np.array_equal(exp["q_assign"][0], exp["q_assign"][1])
    Od = B.sparsepr_dense(Qd, Kd, Vd, wl.softmax_scale)
    for i in range(G * HKV):
        assert_bf16_close(to_np(Od[0, i]), orc.dense_attention(Qs[i], Ks[i // G], Vs[i // G], wl.softmax_scale))


def test_grouped_query_warm_start():
    """A second call over the same scene, seeded with the first call's partitions (one K/V partition per K/V head,
    one query partition per query head), against the oracle's warm-started grouped plan."""
    wl = W.VIDEO_480P.scaled(grid=(3, 30, 52), H=G * HKV, n_probe=64)
    _, _, _, (Q1, K1, V1) = grouped_inputs(wl)
    kw = dict(density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
              softmax_scale=wl.softmax_scale)
    first = B.sparsepr_plan(Q1, K1, V1, **kw)
    e1 = B.sparsepr_plan_export(first)
    # fresh noise around the same tables: noise draws G, G + 1, ... for the queries, draw G for keys and values
    Qs, Ks, Vs = [], [], []
    for kv in range(HKV):
        _, K, V = W.make_head(wl, kv, step=G)
        Ks.append(K)
        Vs.append(V)
        Qs += [W.make_head(wl, kv, step=G + g)[0] for g in range(G)]
    Q2, K2, V2 = [torch.from_numpy(np.stack(x)[None]).to(torch.bfloat16).cuda().contiguous() for x in (Qs, Ks, Vs)]
    kw3 = dict(kw, kmeans_iters=3)
    second = B.sparsepr_plan(Q2, K2, V2, warm_from=first, **kw3)
    assert B.sparsepr_plan_stats(second)["device_error"] == 0
    exp, feat = B.sparsepr_plan_export(second), B.sparsepr_plan_export_features(second)
    prm = orc.default_params(**kw3)
    links = []
    for kv in range(HKV):
        warm = dict(a_K=e1["kv_assign"][kv], a_Q=[e1["q_assign"][kv * G + g] for g in range(G)])
        refs = orc.plan_group(Qs[kv * G:(kv + 1) * G], Ks[kv], prm, kv, kv * G, warm=warm)
        for g in range(G):
            i = kv * G + g
            links.append(plan_links(wl, i, Qs[i], Ks[kv], exp, feat, prm, ref=refs[g], kv=kv,
                                    warm=dict(a_K=warm["a_K"], a_Q=warm["a_Q"][g])))
    check_links(wl, links)
    assert torch.isfinite(B.sparsepr_attend(second, Q2, K2, V2)).all()


def test_grouped_query_needs_the_tensor_core_path():
    Q = torch.randn(1, 4, 256, 64, device="cuda")
    K = torch.randn(1, 2, 256, 64, device="cuda")
    with pytest.raises(B.SparsePRError) as e:
        B.sparsepr_plan(Q, K, K, density=0.5, block=64, n_sample=32, n_probe=8)
    assert e.value.code in (1, 2)
