"""The issued-pairs statistic against a restatement, in Python, of how the block-sparse kernels tile a plan.

128-row tiles per query group over the group's routed K/V groups (16-row boxes, 128-key tiles); remainders of at most
32 rows go to packed tiles instead: 128 rows each, the groups taken in the order (routed K/V groups descending, first
routed group, id), every packed tile streaming the union of its rows' routes."""
import numpy as np
import pytest

from paper_2608_18484_b200 import binding as B
from paper_2608_18484_b200 import workloads as W
from tests.gpu_util import heads_to_device

pytestmark = pytest.mark.gpu

REM_ROWS = 32


def issued_pairs(q_off, kv_off, route_ptr, route_idx):
    nq, nk = np.diff(q_off), np.diff(kv_off)
    boxes = (nk + 15) // 16
    total, order = 0, []
    for a in range(len(nq)):
        r = route_idx[route_ptr[a]:route_ptr[a + 1]]
        kt = (int(boxes[r].sum()) * 16 + 127) // 128
        rem = int(nq[a]) % 128
        if 0 < rem <= REM_ROWS:
            total += (int(nq[a]) // 128) * 128 * kt * 128
            order.append((len(nk) - len(r), int(r[0]) if len(r) else 0, a))
        else:
            total += -(-int(nq[a]) // 128) * 128 * kt * 128
    want, fill = np.zeros(len(nk), bool), 0

    def flush():
        nonlocal total, fill
        total += 128 * ((int(boxes[want].sum()) * 16 + 127) // 128) * 128
        want[:] = False
        fill = 0

    for _, _, a in sorted(order):
        left = int(nq[a]) % 128
        while left > 0:
            take = min(left, 128 - fill)
            want[route_idx[route_ptr[a]:route_ptr[a + 1]]] = True
            fill += take
            left -= take
            if fill == 128:
                flush()
    if fill:
        flush()
    return total


@pytest.mark.parametrize("wl", [W.VIDEO_480P.scaled(grid=(3, 30, 52), H=3), W.WORLD.scaled(grid=(3, 32, 64), H=2)],
                         ids=["480p-like", "world-like"])
def test_issued_pairs_follow_the_documented_tiling(wl):
    heads = list(range(wl.H))
    _, (Qd, Kd, Vd) = heads_to_device(wl, heads)
    plan = B.sparsepr_plan(Qd, Kd, Vd, density=wl.density, block=wl.block, n_sample=wl.n_sample, n_probe=wl.n_probe,
                           softmax_scale=wl.softmax_scale)
    st = B.sparsepr_plan_stats(plan)
    exp = B.sparsepr_plan_export(plan)
    assert st["device_error"] == 0
    want = sum(issued_pairs(np.asarray(exp["q_off"][i]), np.asarray(exp["kv_off"][i]), np.asarray(exp["route_ptr"][i]),
                            np.asarray(exp["route_idx"][i])) for i in range(len(heads)))
    assert st["padded_tile_pairs"] == want
    assert st["padded_tile_pairs"] >= st["routed_pairs"]
