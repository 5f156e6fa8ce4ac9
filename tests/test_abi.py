"""The C-ABI library loads without a GPU and exports every declared symbol; host-side
argument validation and workspace sizing (no kernel is launched here)."""
import ctypes as C
import os
import re

import pytest

from paper_2608_18484_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(B.LIB_PATH):
        from paper_2608_18484_b200 import build
        build.build()
    return B.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sparsepr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sparsepr_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == names


def test_status_strings(lib):
    assert B.status_string(0) == "ok"
    assert len({B.status_string(i) for i in range(7)}) == 7


def _shape(N=4096, d=128, dtype=B.BF16, H=2):
    s = B.Shape(B=1, H=H, N=N, d=d, dv=d, dtype=dtype)
    for f in ("q_stride", "k_stride", "v_stride", "o_stride"):
        getattr(s, f)[:] = [H * N * d, N * d, d]
    return s


def test_workspace_sizes_scale_and_reject(lib):
    p = B.make_params()
    small = lib.sparsepr_plan_workspace_bytes(C.byref(_shape(4096)), C.byref(p))
    big = lib.sparsepr_plan_workspace_bytes(C.byref(_shape(32760, H=24)), C.byref(p))
    assert 0 < small < big < 8 << 30
    att = lib.sparsepr_attend_workspace_bytes(C.byref(_shape(32760, H=24)), C.byref(p))
    assert att >= 3 * 24 * 32760 * 128 * 2                      # group-major copies of Q, K, V
    assert small % 256 == 0 and att % 256 == 0
    # unsupported / invalid shapes and parameters give 0
    assert lib.sparsepr_plan_workspace_bytes(C.byref(_shape(d=96)), C.byref(p)) == 0
    assert lib.sparsepr_plan_workspace_bytes(C.byref(_shape()), C.byref(B.make_params(density=0.0))) == 0
    assert lib.sparsepr_plan_workspace_bytes(C.byref(_shape(N=100)), C.byref(B.make_params(Ck=200))) == 0
    assert lib.sparsepr_plan_workspace_bytes(C.byref(_shape()), C.byref(B.make_params(n_probe=5000))) == 0
    # output rank of the probe-residual subspace: up to 64 eigenvectors, or the full space (no eigenvectors needed)
    assert lib.sparsepr_plan_workspace_bytes(C.byref(_shape()), C.byref(B.make_params(n_probe=128, r_out=100))) == 0
    assert lib.sparsepr_plan_workspace_bytes(C.byref(_shape()), C.byref(B.make_params(n_probe=128, r_out=128))) > 0
    assert lib.sparsepr_plan_workspace_bytes(C.byref(_shape()), C.byref(B.make_params(n_probe=96, r_out=128))) > 0
    assert lib.sparsepr_stage_assign_workspace_bytes(1000, 10, 48) > 1000 * 48 * 4
    assert lib.sparsepr_stage_assign_workspace_bytes(1000, 10, 65) == 0
    # the host-buffer call holds the device copies of Q, K, V, O and one plan + attend workspace per group of heads
    sh = _shape(32760, H=24)
    host = lib.sparsepr_call_host_workspace_bytes(C.byref(sh), C.byref(p), 4)
    assert host >= 4 * 24 * 32760 * 128 * 2 + big + att - (1 << 20) and host % 256 == 0
    assert lib.sparsepr_call_host_workspace_bytes(C.byref(_shape(d=96)), C.byref(p), 4) == 0
    assert lib.sparsepr_call_host_workspace_bytes(C.byref(sh), C.byref(B.make_params(head_offset=-1)), 4) == 0
    assert lib.sparsepr_head_groups(1, 4, 3, 2, None, 0) == 0           # K/V heads must divide the query heads
    assert B.head_groups(1, 24, 24, 4) == [(0, 1, 0, 6), (0, 1, 6, 12), (0, 1, 12, 18), (0, 1, 18, 24)]
    assert B.head_groups(1, 8, 2, 4) == [(0, 1, 0, 4), (0, 1, 4, 8)]     # groups hold whole K/V heads


def test_argument_errors_are_reported_before_any_launch(lib):
    p, s = B.make_params(), _shape()
    h = C.c_void_p()
    assert lib.sparsepr_plan(C.byref(s), C.byref(p), None, None, None, None, 0, None, C.byref(h)) == 1
    bad = _shape(d=96)
    assert lib.sparsepr_plan(C.byref(bad), C.byref(p), 256, 256, None, 256, 1 << 40, None, C.byref(h)) == 2
    assert lib.sparsepr_plan(C.byref(s), C.byref(p), 256, 256, None, None, 0, None, C.byref(h)) == 3      # no workspace
    assert lib.sparsepr_plan(C.byref(s), C.byref(p), 256, 256, None, 256, 1024, None, C.byref(h)) == 3   # too small
    assert lib.sparsepr_plan(C.byref(s), C.byref(p), 256, 256, None, 128, 1 << 40, None, C.byref(h)) == 3  # misaligned
    assert lib.sparsepr_plan_warm(C.byref(s), C.byref(p), 256, 256, None, None, 256, 256, 1 << 40, None, C.byref(h)) == 1
    assert lib.sparsepr_plan_assignments(None, None, None) == 1
    assert lib.sparsepr_attend(None, 256, 256, 256, 256, None, 256, 0, None) == 1
    assert lib.sparsepr_dense(C.byref(s), 0.0, None, 256, 256, 256, None) == 1
    assert lib.sparsepr_dense(C.byref(bad), 0.0, 256, 256, 256, 256, None) == 2
    odd = _shape()
    odd.q_stride[2] = 129                                        # rows not 16-byte aligned
    assert lib.sparsepr_dense(C.byref(odd), 0.0, 256, 256, 256, 256, None) == 2
    assert lib.sparsepr_stage_permute(0, 4, 256, 256, 256, 256, None) == 1
    assert lib.sparsepr_stage_route(4, 5000, 256, 256, 256, 10, 0, 256, 256, 256, None) == 2
    assert lib.sparsepr_stage_assign(10, 4, 70, 256, 256, 256, 256, 1 << 30, None) == 2


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.lib()
