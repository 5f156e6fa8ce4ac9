"""Floating-point parity of the attention path against the oracle, through the C ABI.

Tolerances (from the arithmetic): float32 inputs with float32 accumulation and a
2-ulp exp2 -> relative L2 <= 1e-5; bfloat16 inputs with float32 accumulation and
a bfloat16 output -> relative L2 <= 1e-2 and max-abs <= 2e-2 (one bf16 ulp for elements so large that
rounding the output alone exceeds 2e-2; see tests/gpu_util.py)."""
import numpy as np
import pytest
import torch

from oracle import sparsepr_oracle as orc
from paper_2608_18484_b200 import binding as B
from paper_2608_18484_b200 import workloads as W
from tests.gpu_util import assert_bf16_close, heads_to_device, to_np

pytestmark = pytest.mark.gpu


def oracle_plans(host, prm):
    return [orc.plan_head(Q, K, prm, bh) for bh, (Q, K, V) in enumerate(host)]


def plans_to_host(plans, Cq, Ck):
    return dict(kv_assign=np.stack([p["a_K"] for p in plans]), q_assign=np.stack([p["a_Q"] for p in plans]),
                route_ptr=np.stack([p["route_ptr"] for p in plans]), route_idx=[p["route_idx"] for p in plans],
                probe_idx=np.stack([p["probe_idx"] for p in plans]) if len(plans[0]["probe_idx"]) else None,
                probe_w=np.stack([p["probe_w"] for p in plans]) if len(plans[0]["probe_idx"]) else None)


def check(O, ref, fp32):
    err = orc.rel_l2(O, ref)
    if fp32:
        assert err <= 1e-5, err
    else:
        assert_bf16_close(O, ref)


CASES = [
    ("tiny-f32", W.TINY, dict()),
    ("tiny-f32-ragged", W.TINY.scaled(grid=(3, 31, 29)), dict()),               # N = 2697: ragged tiles everywhere
    ("480p-like-bf16", W.VIDEO_480P.scaled(grid=(3, 30, 52), H=2, n_probe=64), dict()),
    ("world-like-bf16", W.WORLD.scaled(grid=(3, 32, 64), H=2, n_probe=96), dict()),
    ("720p-like-bf16", W.VIDEO_720P.scaled(grid=(2, 45, 80), H=2, n_probe=64), dict()),
    ("480p-like-bf16-sparser", W.VIDEO_480P.scaled(grid=(3, 30, 52), H=2, n_probe=64, density=0.12), dict()),
    ("480p-like-bf16-denser", W.VIDEO_480P.scaled(grid=(3, 30, 52), H=2, n_probe=64, density=0.35), dict(r_out=128)),
    # output rank r = min(r_out, M, d_v) above the 64 eigenvectors the solver delivers: the projector is the identity
    ("480p-like-bf16-full-rank", W.VIDEO_480P.scaled(grid=(3, 30, 52), H=2, n_probe=128), dict(r_out=128)),
    ("480p-like-bf16-rank-96", W.VIDEO_480P.scaled(grid=(3, 30, 52), H=2, n_probe=96), dict(r_out=128, lam=10.0)),
    # 38 key tiles over 9 probe slices of 5 tiles: the last slice is empty and must not contribute
    ("480p-like-bf16-empty-probe-slice", W.VIDEO_480P.scaled(grid=(3, 30, 53), H=2, n_probe=64), dict()),
]


@pytest.mark.parametrize("name,wl,extra", CASES, ids=[c[0] for c in CASES])
def test_attend_on_injected_oracle_plan(name, wl, extra):
    heads = list(range(min(wl.H, 2)))
    host, (Qd, Kd, Vd) = heads_to_device(wl, heads)
    # the workspaces come from the caching allocator: leave NaN behind so that anything read before it is written shows
    junk = torch.full((64 << 20,), float("nan"), device="cuda")
    del junk
    kw = dict(density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
              softmax_scale=wl.softmax_scale, **extra)
    prm = orc.default_params(**kw)
    plans = oracle_plans(host, prm)
    C = -(-wl.N // wl.block)
    plan = B.sparsepr_plan_import(Qd, Kd, Vd, plans_to_host(plans, C, C), **kw)
    O, Osp = B.sparsepr_attend(plan, Qd, Kd, Vd, return_sparse=True)
    st = B.sparsepr_plan_stats(plan)
    assert st["device_error"] == 0
    assert st["routed_pairs"] == sum(p["routed_pairs"] for p in plans)
    exp = B.sparsepr_plan_export(plan)
    fp32 = wl.dtype == "f32"
    for i, (Q, K, V) in enumerate(host):
        assert np.array_equal(exp["kv_perm"][i], plans[i]["kv_perm"]) and np.array_equal(exp["q_off"][i], plans[i]["q_off"])
        O_hat, O_sp, fit = orc.attend_head(Q, K, V, plans[i], prm)
        check(to_np(Osp[0, i]), O_sp, True if fp32 else False)
        check(to_np(O[0, i]), O_hat, fp32)
        # probe rows carry the exact output
        P = plans[i]["probe_idx"]
        check(to_np(O[0, i])[P], orc.dense_attention(Q, K, V, plans[i]["scale"], rows=P), fp32)


def test_hard_drop_mode_and_full_density():
    wl = W.TINY.scaled(grid=(2, 32, 32))
    host, (Qd, Kd, Vd) = heads_to_device(wl, [0, 1])
    kw = dict(density=0.25, block=64, n_sample=64, n_probe=32, softmax_scale=1.0, mode=1)
    prm = orc.default_params(**kw)
    plans = oracle_plans(host, prm)
    plan = B.sparsepr_plan_import(Qd, Kd, Vd, plans_to_host(plans, 32, 32), **kw)
    O = B.sparsepr_attend(plan, Qd, Kd, Vd)
    for i, (Q, K, V) in enumerate(host):
        check(to_np(O[0, i]), orc.attend_head(Q, K, V, plans[i], prm)[0], True)
    # density >= 1: every cell routed -> dense attention, through the GPU's own plan
    plan = B.sparsepr_plan(Qd, Kd, Vd, density=1.0, block=64, n_sample=64, n_probe=32, softmax_scale=1.0)
    O = B.sparsepr_attend(plan, Qd, Kd, Vd)
    st = B.sparsepr_plan_stats(plan)
    assert st["routed_pairs"] == 2 * wl.N * wl.N and st["device_error"] == 0
    for i, (Q, K, V) in enumerate(host):
        check(to_np(O[0, i]), orc.dense_attention(Q, K, V, 1.0), True)


@pytest.mark.parametrize("dtype,N,d", [("f32", 1000, 64), ("bf16", 1111, 128), ("f32", 64, 128), ("bf16", 4100, 64)])
def test_dense_entry_point(dtype, N, d):
    rng = np.random.default_rng(N)
    Q, K, V = [rng.normal(size=(N, d)).astype(np.float32) * s for s in (d ** -0.25, d ** -0.25, 1.0)]
    if dtype == "bf16":
        Q, K, V = W.round_to_bf16(Q), W.round_to_bf16(K), W.round_to_bf16(V)
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    Qd, Kd, Vd = [torch.from_numpy(x)[None, None].to(dt).cuda() for x in (Q, K, V)]
    O = B.sparsepr_dense(Qd, Kd, Vd, 1.0)
    check(to_np(O[0, 0]), orc.dense_attention(Q, K, V, 1.0), dtype == "f32")
    O0 = B.sparsepr_dense(Qd, Kd, Vd, 0.0)                       # default scale 1/sqrt(d)
    check(to_np(O0[0, 0]), orc.dense_attention(Q, K, V, d ** -0.5), dtype == "f32")


def test_strided_layout_bnhd():
    """[B, N, H, d] storage viewed as [B, H, N, d]: head stride d, token stride H*d."""
    wl = W.TINY.scaled(grid=(1, 32, 32))
    host, (Qd, Kd, Vd) = heads_to_device(wl, [0, 1])
    Qs, Ks, Vs = [x.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for x in (Qd, Kd, Vd)]
    assert Qs.stride(1) == 64 and Qs.stride(2) == 128
    O = B.sparsepr_dense(Qs, Ks, Vs, 1.0)
    assert O.stride() == Qs.stride()
    for i, (Q, K, V) in enumerate(host):
        check(to_np(O[0, i]), orc.dense_attention(Q, K, V, 1.0), True)
    kw = dict(density=0.3, block=64, n_sample=64, n_probe=16, softmax_scale=1.0)
    p1 = B.sparsepr_plan(Qs, Ks, Vs, **kw)
    p2 = B.sparsepr_plan(Qd, Kd, Vd, **kw)
    e1, e2 = B.sparsepr_plan_export(p1), B.sparsepr_plan_export(p2)
    for k in e1:                                                # the plan does not depend on the memory layout
        if k == "route_idx":                                    # only the first route_ptr[-1] entries of a slab are defined
            for i in range(2):
                n = e1["route_ptr"][i][-1]
                assert np.array_equal(e1[k][i][:n], e2[k][i][:n])
        else:
            assert np.array_equal(e1[k], e2[k]), k
    assert torch.equal(B.sparsepr_attend(p1, Qs, Ks, Vs), B.sparsepr_attend(p2, Qd, Kd, Vd))
