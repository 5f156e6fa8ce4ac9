"""The host-buffer call: a problem is cut into groups of heads that are uploaded, computed and downloaded as a
pipeline.  Every group is a call of its own whose `head_offset` names its first head, so the deterministic row
samples (sampled queries of Appendix B.1, k-means initialisation) stay those of the whole problem: the plan of a
group must equal, bit for bit, the rows of the plan of one call over all heads.  The outputs agree up to the
summation order of the probe rows (the number of key slices they are summed over is chosen per call from the head
count); with one group they are identical."""
import numpy as np
import pytest
import torch

from paper_2608_18484_b200 import binding as B
from paper_2608_18484_b200 import workloads as W
from tests.gpu_util import heads_to_device


def test_head_groups_cover_every_head_once():
    for Bn, H, G, groups in [(1, 24, 1, 4), (1, 24, 1, 5), (1, 4, 2, 4), (2, 6, 2, 3), (4, 8, 1, 2), (3, 2, 1, 8),
                             (1, 1, 1, 4), (2, 40, 8, 7)]:
        boxes = B.head_groups(Bn, H, H // G, groups)
        seen = np.zeros((Bn, H), dtype=int)
        last = -1
        for (b0, b1, h0, h1) in boxes:
            assert 0 <= b0 < b1 <= Bn and 0 <= h0 < h1 <= H and h0 % G == 0 and h1 % G == 0
            assert b1 - b0 == 1 or (h0, h1) == (0, H)          # heads b H + h of a box are consecutive
            assert b0 * H + h0 == last + 1                        # boxes follow each other in that order
            last = (b1 - 1) * H + h1 - 1
            seen[b0:b1, h0:h1] += 1
        assert (seen == 1).all(), (Bn, H, G, groups)
        assert len(boxes) <= groups + Bn


def _pinned(t):
    return t.cpu().pin_memory()


@pytest.mark.gpu
@pytest.mark.parametrize("name,wl", [("tiny-f32", W.TINY.scaled(H=4)),
                                     ("480p-like-bf16", W.VIDEO_480P.scaled(grid=(3, 30, 52), H=4, n_probe=64))],
                         ids=["tiny-f32", "480p-like-bf16"])
def test_pipelined_host_call_equals_one_device_call(name, wl):
    _, (Qd, Kd, Vd) = heads_to_device(wl, [0, 1, 2, 3])
    params = B.make_params(density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
                           softmax_scale=wl.softmax_scale, seed=5)
    plan = B.sparsepr_plan(Qd, Kd, Vd, params=params)
    ref = B.sparsepr_attend(plan, Qd, Kd, Vd).cpu()
    assert B.sparsepr_plan_stats(plan)["device_error"] == 0
    full = B.sparsepr_plan_export(plan)
    # a group of heads with its offset reproduces its rows of the whole plan
    prm2 = B.Params.from_buffer_copy(params)
    prm2.head_offset = 2
    part = B.sparsepr_plan_export(B.sparsepr_plan(Qd[:, 2:], Kd[:, 2:], Vd[:, 2:], params=prm2))
    for key in ("kv_assign", "q_assign", "kv_perm", "q_perm", "route_ptr", "probe_idx", "probe_w"):
        assert np.array_equal(np.asarray(part[key]), np.asarray(full[key])[2:]), key
    for i in range(2):                                              # CSR column lists: the used part of every head
        n = int(part["route_ptr"][i][-1])
        assert np.array_equal(part["route_idx"][i][:n], full["route_idx"][2 + i][:n])
    Qh, Kh, Vh = _pinned(Qd), _pinned(Kd), _pinned(Vd)
    tol = 1e-5 if wl.dtype == "f32" else 2.0 ** -7
    for groups in (1, 2, 3, 4):
        Oh = torch.full(Qh.shape, float("nan"), dtype=Qh.dtype).pin_memory()
        B.sparsepr_call_host(Qh, Kh, Vh, Oh, params, groups=groups)
        if groups == 1:
            assert torch.equal(Oh, ref)
        diff = (Oh.float() - ref.float()).abs()
        assert bool((diff <= tol * (1.0 + ref.float().abs())).all()), (groups, float(diff.max()))
    # the samples really depend on the head index: the heads of the second half, taken as a problem of their own
    # without the offset, come out differently
    other = B.sparsepr_plan_export(B.sparsepr_plan(Qd[:, 2:], Kd[:, 2:], Vd[:, 2:], params=params))
    assert not np.array_equal(np.asarray(other["kv_assign"]), np.asarray(full["kv_assign"])[2:])


@pytest.mark.gpu
def test_pipelined_host_call_over_batches_and_shared_kv_heads():
    wl = W.VIDEO_480P.scaled(grid=(3, 30, 52), H=4, n_probe=64)
    _, (Qd, Kd, Vd) = heads_to_device(wl, [0, 1, 2, 3])
    params = B.make_params(density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
                           softmax_scale=wl.softmax_scale)
    # two batch entries of two heads each
    Q2, K2, V2 = (t.reshape(2, 2, *t.shape[2:]).contiguous() for t in (Qd, Kd, Vd))
    ref = B.sparsepr_attend(B.sparsepr_plan(Q2, K2, V2, params=params), Q2, K2, V2).cpu()
    def close(Oh, ref):
        diff = (Oh.float() - ref.float()).abs()
        return bool((diff <= 2.0 ** -7 * (1.0 + ref.float().abs())).all())

    for groups in (2, 4):
        Oh = torch.full(Q2.shape, float("nan"), dtype=Q2.dtype).pin_memory()
        B.sparsepr_call_host(_pinned(Q2), _pinned(K2), _pinned(V2), Oh, params, groups=groups)
        assert close(Oh, ref), groups
    # grouped-query attention: four query heads on two K/V heads; groups hold whole K/V heads
    Kg, Vg = Kd[:, :2].contiguous(), Vd[:, :2].contiguous()
    ref = B.sparsepr_attend(B.sparsepr_plan(Qd, Kg, Vg, params=params), Qd, Kg, Vg).cpu()
    Oh = torch.full(Qd.shape, float("nan"), dtype=Qd.dtype).pin_memory()
    B.sparsepr_call_host(_pinned(Qd), _pinned(Kg), _pinned(Vg), Oh, params, groups=4)
    assert close(Oh, ref)
    bad = B.make_params(density=wl.density, head_offset=1)
    with pytest.raises(B.SparsePRError):
        B.sparsepr_plan(Qd, Kg, Vg, params=bad)
