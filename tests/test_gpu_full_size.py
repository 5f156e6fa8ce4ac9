"""Parity at the full size of the bench workload, on sampled output rows.

The whole call runs on the GPU exactly as bench.py launches it (video-dit-480p-like:
N = 32760, d = 128, bf16; four heads keep host memory and the oracle's time small).
The oracle then evaluates, for the GPU's own plan, a sample of output rows one by
one: ordinary rows, rows of short group remainders (handled by the remainder kernel),
first rows of 128-row tiles, and probe rows.  Properties that hold at any size are
checked on every head."""
import numpy as np
import pytest
import torch

from oracle import sparsepr_oracle as orc
from paper_2608_18484_b200 import binding as B
from paper_2608_18484_b200 import workloads as W
from tests.gpu_util import assert_bf16_close, heads_to_device, to_np

pytestmark = pytest.mark.gpu


def test_full_size_480p_sampled_rows():
    wl = W.VIDEO_480P.scaled(H=4)
    heads = [0, 1, 2, 3]
    host, (Qd, Kd, Vd) = heads_to_device(wl, heads)
    kw = dict(density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
              softmax_scale=wl.softmax_scale)
    plan = B.sparsepr_plan(Qd, Kd, Vd, **kw)
    O, Osp = B.sparsepr_attend(plan, Qd, Kd, Vd, return_sparse=True)
    st = B.sparsepr_plan_stats(plan)
    exp = B.sparsepr_plan_export(plan)
    assert st["device_error"] == 0
    assert torch.isfinite(O).all()
    prm = orc.default_params(**kw)
    C = -(-wl.N // wl.block)
    budget = orc.pair_budget(wl.density, wl.N, wl.N, wl.n_probe)
    rng = np.random.default_rng(7)
    for i in heads:
        aK, aQ = exp["kv_assign"][i], exp["q_assign"][i]
        ptr, idx = exp["route_ptr"][i], exp["route_idx"][i]
        n_q, n_k = np.bincount(aQ, minlength=C), np.bincount(aK, minlength=C)
        # properties at any size: permutations, budget, probes
        p0, _, o0 = orc.group_permutation(aQ, C)
        assert np.array_equal(exp["q_perm"][i], p0) and np.array_equal(exp["q_off"][i], o0)
        pairs = orc.routed_pairs(n_q, n_k, ptr, idx[:ptr[-1]])
        assert pairs == exp["routed_pairs"][i] and pairs <= budget
        assert len(set(exp["probe_idx"][i].tolist())) == wl.n_probe
    # sampled rows against the oracle's evaluation of the GPU plan (head 0 and the last head)
    for i in (0, 3):
        Q, K, V = host[i]
        aK, aQ = exp["kv_assign"][i], exp["q_assign"][i]
        ptr, idx = exp["route_ptr"][i], exp["route_idx"][i]
        P = exp["probe_idx"][i]
        gplan = dict(scale=wl.softmax_scale, a_Q=aQ, a_K=aK, route_ptr=ptr, route_idx=idx[:ptr[-1]], probe_idx=P,
                     M=len(P), probe_w=exp["probe_w"][i].astype(np.float64))
        q_perm, q_off = exp["q_perm"][i], exp["q_off"][i]
        sizes = np.diff(q_off)
        rows = list(rng.choice(wl.N, 24, replace=False))
        small = [a for a in range(C) if 0 < sizes[a] % 128 <= 32]      # remainders packed across groups
        mid = [a for a in range(C) if sizes[a] % 128 > 32]              # remainders with a (partly empty) tile of their own
        assert small and mid, "the workload is expected to leave short and long remainders"
        for a in small[:6] + mid[:3]:                           # last row of the remainder, first row of the group
            rows += [int(q_perm[q_off[a + 1] - 1]), int(q_perm[q_off[a]])]
        rows += [int(p) for p in P[:4]]
        rows = np.array(sorted(set(rows)), dtype=np.int64)
        O_hat, O_sp, _ = orc.attend_head(Q, K, V, gplan, prm, rows=rows)
        got, got_sp = to_np(O[0, i])[rows], to_np(Osp[0, i])[rows]
        assert_bf16_close(got_sp, O_sp)
        assert_bf16_close(got, O_hat)


@pytest.mark.parametrize("wl", [W.WORLD.scaled(H=2), W.VIDEO_720P.scaled(H=1)], ids=["world-like", "720p-like"])
def test_more_than_256_groups_sampled_rows(wl):
    """world-model-like and video-dit-720p-like at full length (N = 49152 / 75600, 384 / 591 groups per side): the
    k-means assignment streams the centroids in two / three chunks of 256 per row tile (the last one partly filled)
    and the attention kernels see more groups than one chunk holds.  Properties on every head, sampled rows of the
    GPU's own plan against the oracle on the first."""
    heads = list(range(wl.H))
    host, (Qd, Kd, Vd) = heads_to_device(wl, heads)
    kw = dict(density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
              softmax_scale=wl.softmax_scale)
    plan = B.sparsepr_plan(Qd, Kd, Vd, **kw)
    O, Osp = B.sparsepr_attend(plan, Qd, Kd, Vd, return_sparse=True)
    st = B.sparsepr_plan_stats(plan)
    exp = B.sparsepr_plan_export(plan)
    assert st["device_error"] == 0
    assert torch.isfinite(O).all()
    prm = orc.default_params(**kw)
    C = -(-wl.N // wl.block)
    assert C > 256
    budget = orc.pair_budget(wl.density, wl.N, wl.N, wl.n_probe)
    rng = np.random.default_rng(11)
    for i in heads:
        aK, aQ = exp["kv_assign"][i], exp["q_assign"][i]
        ptr, idx = exp["route_ptr"][i], exp["route_idx"][i]
        n_q, n_k = np.bincount(aQ, minlength=C), np.bincount(aK, minlength=C)
        assert aK.min() >= 0 and aK.max() < C and aQ.min() >= 0 and aQ.max() < C
        assert (n_k > 0).sum() > 256 and (n_q > 0).sum() > 256        # groups of both chunks are in use
        p0, _, o0 = orc.group_permutation(aK, C)
        assert np.array_equal(exp["kv_perm"][i], p0) and np.array_equal(exp["kv_off"][i], o0)
        p0, _, o0 = orc.group_permutation(aQ, C)
        assert np.array_equal(exp["q_perm"][i], p0) and np.array_equal(exp["q_off"][i], o0)
        pairs = orc.routed_pairs(n_q, n_k, ptr, idx[:ptr[-1]])
        assert pairs == exp["routed_pairs"][i] and pairs <= budget
        assert len(set(exp["probe_idx"][i].tolist())) == wl.n_probe
    Q, K, V = host[0]
    P = exp["probe_idx"][0]
    gplan = dict(scale=wl.softmax_scale, a_Q=exp["q_assign"][0], a_K=exp["kv_assign"][0], route_ptr=exp["route_ptr"][0],
                 route_idx=exp["route_idx"][0][:exp["route_ptr"][0][-1]], probe_idx=P, M=len(P),
                 probe_w=exp["probe_w"][0].astype(np.float64))
    rows = np.array(sorted(set(list(rng.choice(wl.N, 24, replace=False)) + [int(p) for p in P[:4]])), dtype=np.int64)
    O_hat, O_sp, _ = orc.attend_head(Q, K, V, gplan, prm, rows=rows)
    got, got_sp = to_np(O[0, 0])[rows], to_np(Osp[0, 0])[rows]
    assert_bf16_close(got_sp, O_sp)
    assert_bf16_close(got, O_hat)


def test_reconstruction_error_matches_the_oracle_at_scale():
    """The whole call of the oracle and of the GPU on the same bytes at a non-toy size (head 0 of the 480p-like
    workload, 16 of 21 frames, N = 24960, 195 groups per side): the two plans are built independently (float64 vs
    float32, so single near-tie decisions may differ), and what has to agree is the reconstruction error against
    float64 exact attention, with and without the probe repair, and the realised density."""
    wl = W.VIDEO_480P.scaled(grid=(16, 30, 52), H=1)
    host, (Qd, Kd, Vd) = heads_to_device(wl, [0])
    Q, K, V = host[0]
    kw = dict(density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
              softmax_scale=wl.softmax_scale)
    plan = B.sparsepr_plan(Qd, Kd, Vd, **kw)
    O, Osp = B.sparsepr_attend(plan, Qd, Kd, Vd, return_sparse=True)
    st = B.sparsepr_plan_stats(plan)
    assert st["device_error"] == 0
    prm = orc.default_params(**kw)
    O_ref, O_ref_sp, ref, _ = orc.sparsepr_head(Q, K, V, prm, 0)
    exact = orc.dense_attention(Q, K, V, wl.softmax_scale)
    e_gpu, e_orc = orc.rel_l2(to_np(O[0, 0]), exact), orc.rel_l2(O_ref, exact)
    h_gpu, h_orc = orc.rel_l2(to_np(Osp[0, 0]), exact), orc.rel_l2(O_ref_sp, exact)
    # bf16 output rounding alone is 1.7e-3 relative; the errors themselves are about 0.1
    assert abs(e_gpu - e_orc) <= 2e-3 and abs(h_gpu - h_orc) <= 2e-3, (e_gpu, e_orc, h_gpu, h_orc)
    assert abs(st["rho_route"] - ref["rho_route"]) <= 1e-3
    assert (B.sparsepr_plan_export(plan)["kv_assign"][0] == ref["a_K"]).mean() >= 0.97
