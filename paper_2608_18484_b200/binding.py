"""Thin ctypes binding of libsparsepr.so (the C ABI declared in include/sparsepr.h).

Only argument marshalling happens here: PyTorch supplies device memory and the
current CUDA stream, every step of the computation runs inside the library.
There is no fallback: if the library is missing the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsparsepr.so")
_lib = None

OK = 0
F32, BF16 = 0, 1
STATUS = {0: "OK", 1: "ERR_INVALID_ARG", 2: "ERR_UNSUPPORTED", 3: "ERR_WORKSPACE", 4: "ERR_CUDA",
          5: "ERR_NUMERIC", 6: "ERR_TIMEOUT"}


class SparsePRError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__("%s failed: %s (%s)" % (where, STATUS.get(code, code), status_string(code)))


class Shape(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("N", C.c_int32), ("d", C.c_int32), ("dv", C.c_int32),
                ("dtype", C.c_int32), ("q_stride", C.c_int64 * 3), ("k_stride", C.c_int64 * 3),
                ("v_stride", C.c_int64 * 3), ("o_stride", C.c_int64 * 3), ("Hkv", C.c_int32)]


class Params(C.Structure):
    _fields_ = [("density", C.c_float), ("block", C.c_int32), ("Ck", C.c_int32), ("Cq", C.c_int32),
                ("n_sample", C.c_int32), ("n_probe", C.c_int32), ("rK", C.c_int32), ("rQ", C.c_int32),
                ("r_out", C.c_int32), ("lam", C.c_float), ("eps_rms", C.c_float), ("eps_std", C.c_float),
                ("kmeans_iters", C.c_int32), ("softmax_scale", C.c_float), ("seed", C.c_uint64), ("mode", C.c_int32),
                ("partition", C.c_int32), ("head_offset", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("routed_pairs", C.c_int64), ("routed_cells", C.c_int64), ("padded_tile_pairs", C.c_int64),
                ("rho_route", C.c_double), ("rho_exec", C.c_double), ("rho_route_min", C.c_double),
                ("rho_route_max", C.c_double), ("nonempty_kv_groups_min", C.c_int32),
                ("nonempty_q_groups_min", C.c_int32), ("max_kv_group", C.c_int32), ("max_q_group", C.c_int32),
                ("assign_rechecked_rows", C.c_int32), ("device_error", C.c_int32),
                ("kmeans_passes_kv", C.c_int32), ("kmeans_passes_q", C.c_int32)]


class PlanHost(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("kv_assign", "q_assign", "kv_perm", "q_perm", "kv_off", "q_off",
                                            "route_ptr", "route_idx", "probe_idx", "probe_w", "routed_pairs")]


class PlanFeatures(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("F_K", "F_Q", "phi_Q", "kappa", "theta", "score")]


STAGES = ["key_metric", "key_project", "key_kmeans", "key_permute", "query_metric", "query_project", "query_kmeans",
          "query_permute", "probe_select", "route", "gather", "probe_rows", "fit", "attention", "correction", "probe_write", "dense"]


class Profile(C.Structure):
    _fields_ = [("ms", C.c_float * len(STAGES))]

    def as_dict(self):
        return {n: float(self.ms[i]) for i, n in enumerate(STAGES)}


EXPORTS = ["sparsepr_stage_assign_static", "sparsepr_plan_timed", "sparsepr_attend_timed", "sparsepr_dense_timed", "sparsepr_status_string", "sparsepr_plan_workspace_bytes", "sparsepr_attend_workspace_bytes",
           "sparsepr_plan", "sparsepr_attend", "sparsepr_dense", "sparsepr_plan_stats", "sparsepr_plan_export",
           "sparsepr_plan_export_features", "sparsepr_plan_warm", "sparsepr_plan_assignments",
           "sparsepr_selftest_bounded_wait", "sparsepr_call_host", "sparsepr_call_host_workspace_bytes",
           "sparsepr_head_groups", "sparsepr_plan_device_error",
           "sparsepr_plan_import", "sparsepr_plan_destroy", "sparsepr_stage_assign_workspace_bytes",
           "sparsepr_stage_assign", "sparsepr_stage_permute", "sparsepr_stage_route"]


def lib():
    """Loads the CUDA library on first use; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libsparsepr.so is missing: run `python -m paper_2608_18484_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(LIB_PATH)
        vp, sz, i32, i64 = C.c_void_p, C.c_size_t, C.c_int32, C.c_int64
        L.sparsepr_status_string.restype = C.c_char_p
        L.sparsepr_status_string.argtypes = [C.c_int]
        for f in (L.sparsepr_plan_workspace_bytes, L.sparsepr_attend_workspace_bytes):
            f.restype = sz
            f.argtypes = [C.POINTER(Shape), C.POINTER(Params)]
        L.sparsepr_plan.argtypes = [C.POINTER(Shape), C.POINTER(Params), vp, vp, vp, vp, sz, vp, C.POINTER(vp)]
        L.sparsepr_attend.argtypes = [vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.sparsepr_dense.argtypes = [C.POINTER(Shape), C.c_float, vp, vp, vp, vp, vp]
        L.sparsepr_plan_timed.argtypes = L.sparsepr_plan.argtypes + [C.POINTER(Profile)]
        L.sparsepr_plan_warm.argtypes = [C.POINTER(Shape), C.POINTER(Params), vp, vp, vp, vp, vp, vp, sz, vp, C.POINTER(vp)]
        L.sparsepr_plan_assignments.argtypes = [vp, C.POINTER(vp), C.POINTER(vp)]
        L.sparsepr_selftest_bounded_wait.argtypes = [vp, vp]
        L.sparsepr_attend_timed.argtypes = L.sparsepr_attend.argtypes + [C.POINTER(Profile)]
        L.sparsepr_dense_timed.argtypes = L.sparsepr_dense.argtypes + [C.POINTER(Profile)]
        L.sparsepr_plan_stats.argtypes = [vp, C.POINTER(Stats)]
        L.sparsepr_plan_export.argtypes = [vp, C.POINTER(PlanHost)]
        L.sparsepr_plan_export_features.argtypes = [vp, C.POINTER(PlanFeatures)]
        L.sparsepr_plan_import.argtypes = [C.POINTER(Shape), C.POINTER(Params), C.POINTER(PlanHost), vp, sz, vp,
                                           C.POINTER(vp)]
        L.sparsepr_call_host_workspace_bytes.restype = sz
        L.sparsepr_call_host_workspace_bytes.argtypes = [C.POINTER(Shape), C.POINTER(Params), i32]
        L.sparsepr_call_host.argtypes = [C.POINTER(Shape), C.POINTER(Params), vp, vp, vp, vp, i32, vp, sz, vp]
        L.sparsepr_head_groups.restype = i32
        L.sparsepr_head_groups.argtypes = [i32, i32, i32, i32, C.POINTER(i32), i32]
        L.sparsepr_plan_device_error.argtypes = [vp, C.POINTER(i32)]
        L.sparsepr_plan_destroy.argtypes = [vp]
        L.sparsepr_plan_destroy.restype = None
        L.sparsepr_stage_assign_workspace_bytes.restype = sz
        L.sparsepr_stage_assign_workspace_bytes.argtypes = [i32, i32, i32]
        L.sparsepr_stage_assign.argtypes = [i32, i32, i32, vp, vp, vp, vp, sz, vp]
        L.sparsepr_stage_assign_static.argtypes = [i32, i32, i32, vp, vp, vp, vp]
        L.sparsepr_stage_permute.argtypes = [i32, i32, vp, vp, vp, vp, vp]
        L.sparsepr_stage_route.argtypes = [i32, i32, vp, vp, vp, i64, i32, vp, vp, vp, vp]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().sparsepr_status_string(int(code)).decode()


def _check(code, where):
    if code != OK:
        raise SparsePRError(code, where)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("Q, K, V must be float32 or bfloat16")


def make_shape(Q, K, V, O) -> Shape:
    for t in (Q, K, V, O):
        if t.dim() != 4 or not t.is_cuda or t.stride(3) != 1:
            raise ValueError("expected CUDA tensors [B, H, N, d] with a contiguous last dimension")
    B, H, N, d = Q.shape
    if K.shape[1] != V.shape[1] or H % K.shape[1] != 0:
        raise ValueError("K and V need the same number of heads, a divisor of the number of query heads")
    s = Shape(B=B, H=H, N=N, d=d, dv=V.shape[3], dtype=_dtype_code(Q), Hkv=K.shape[1])
    for name, t in (("q_stride", Q), ("k_stride", K), ("v_stride", V), ("o_stride", O)):
        getattr(s, name)[:] = [t.stride(0), t.stride(1), t.stride(2)]
    return s


def make_params(density=0.25, block=128, Ck=0, Cq=0, n_sample=256, n_probe=128, rK=48, rQ=64, r_out=16, lam=0.1,
                eps_rms=1e-6, eps_std=1e-6, kmeans_iters=8, softmax_scale=0.0, seed=0, mode=0, partition=0,
                head_offset=0) -> Params:
    return Params(partition=partition, head_offset=head_offset, density=density, block=block, Ck=Ck, Cq=Cq, n_sample=n_sample, n_probe=n_probe, rK=rK, rQ=rQ,
                  r_out=r_out, lam=lam, eps_rms=eps_rms, eps_std=eps_std, kmeans_iters=kmeans_iters,
                  softmax_scale=softmax_scale, seed=seed, mode=mode)


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


class Plan:
    """Owns the host handle and the device workspace a plan lives in."""

    def __init__(self, handle, workspace, shape: Shape, params: Params, attend_bytes: int):
        self.handle, self.workspace, self.shape, self.params = handle, workspace, shape, params
        self.attend_bytes = attend_bytes
        self.attend_workspace = None

    @property
    def BH(self):
        return self.shape.B * self.shape.H

    @property
    def BHkv(self):
        return self.shape.B * (self.shape.Hkv or self.shape.H)

    @property
    def groups(self):
        blk = self.params.block or 128
        n = -(-self.shape.N // blk)
        return (self.params.Ck or n, self.params.Cq or n)

    @property
    def M(self):
        return 0 if self.params.mode == 1 else min(self.params.n_probe, self.shape.N)

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.sparsepr_plan_destroy(self.handle)
            self.handle = None


def sparsepr_plan(Q, K, V=None, params: Params | None = None, profile: Profile | None = None,
                  warm_from: "Plan | None" = None, **kw) -> Plan:
    """Stages 1-2: partition, permutations, probe set and routes for every head.
    With `profile` the timed entry point is used and per-stage milliseconds are added to it.
    With `warm_from` (an earlier plan over the same token grid) both k-means runs start from that plan's partition."""
    params = params or make_params(**kw)
    shape = make_shape(Q, K, K if V is None else V, Q)
    L = lib()
    nbytes = L.sparsepr_plan_workspace_bytes(C.byref(shape), C.byref(params))
    if nbytes == 0:
        raise SparsePRError(1, "sparsepr_plan_workspace_bytes")
    ws = _workspace(nbytes, Q.device)
    handle = C.c_void_p()
    args = (C.byref(shape), C.byref(params), Q.data_ptr(), K.data_ptr(), None if V is None else V.data_ptr(),
            ws.data_ptr(), ws.numel(), _stream(), C.byref(handle))
    keep = None
    if warm_from is not None:
        if profile is not None:
            raise ValueError("the warm-started plan has no timed variant")
        pk, pq = C.c_void_p(), C.c_void_p()
        _check(L.sparsepr_plan_assignments(warm_from.handle, C.byref(pk), C.byref(pq)), "sparsepr_plan_assignments")
        _check(L.sparsepr_plan_warm(*args[:5], pk, pq, *args[5:]), "sparsepr_plan_warm")
        keep = warm_from.workspace                   # read by queued work: keep the earlier workspace alive with this plan
    elif profile is None:
        _check(L.sparsepr_plan(*args), "sparsepr_plan")
    else:
        _check(L.sparsepr_plan_timed(*args, C.byref(profile)), "sparsepr_plan_timed")
    plan = Plan(handle, ws, shape, params, L.sparsepr_attend_workspace_bytes(C.byref(shape), C.byref(params)))
    plan.warm_source = keep
    return plan


def sparsepr_attend(plan: Plan, Q, K, V, out=None, return_sparse=False, profile: Profile | None = None):
    """Stages 3-4: block-sparse attention, probe rows, fit and corrected output."""
    O = torch.empty_like(Q) if out is None else out
    shape = make_shape(Q, K, V, O)
    for f in ("q_stride", "k_stride", "v_stride", "o_stride"):
        if list(getattr(shape, f)) != list(getattr(plan.shape, f)):
            raise ValueError("tensor strides differ from the ones the plan was built for")
    if plan.attend_workspace is None:
        plan.attend_workspace = _workspace(plan.attend_bytes, Q.device)
    ws = plan.attend_workspace
    Osp = torch.empty(Q.shape, dtype=torch.float32, device=Q.device) if return_sparse else None
    args = (plan.handle, Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(),
            None if Osp is None else Osp.data_ptr(), ws.data_ptr(), ws.numel(), _stream())
    if profile is None:
        _check(lib().sparsepr_attend(*args), "sparsepr_attend")
    else:
        _check(lib().sparsepr_attend_timed(*args, C.byref(profile)), "sparsepr_attend_timed")
    return (O, Osp) if return_sparse else O


def sparsepr_dense(Q, K, V, softmax_scale=0.0, out=None, profile: Profile | None = None):
    """Dense attention, Eq. 1, by the same build's kernels."""
    O = torch.empty_like(Q) if out is None else out
    shape = make_shape(Q, K, V, O)
    args = (C.byref(shape), float(softmax_scale), Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), _stream())
    if profile is None:
        _check(lib().sparsepr_dense(*args), "sparsepr_dense")
    else:
        _check(lib().sparsepr_dense_timed(*args, C.byref(profile)), "sparsepr_dense_timed")
    return O


def sparsepr_plan_stats(plan: Plan) -> dict:
    st = Stats()
    _check(lib().sparsepr_plan_stats(plan.handle, C.byref(st)), "sparsepr_plan_stats")
    return {n: getattr(st, n) for n, _ in Stats._fields_}


def _host_arrays(plan: Plan) -> dict:
    BH, N, BHkv = plan.BH, plan.shape.N, plan.BHkv
    Ck, Cq = plan.groups
    M = max(plan.M, 1)
    return dict(kv_assign=np.empty((BHkv, N), np.int32), q_assign=np.empty((BH, N), np.int32),
                kv_perm=np.empty((BHkv, N), np.int32), q_perm=np.empty((BH, N), np.int32),
                kv_off=np.empty((BHkv, Ck + 1), np.int32), q_off=np.empty((BH, Cq + 1), np.int32),
                route_ptr=np.empty((BH, Cq + 1), np.int32), route_idx=np.empty((BH, Cq * Ck), np.int32),
                probe_idx=np.empty((BH, M), np.int32), probe_w=np.empty((BH, M), np.float32),
                routed_pairs=np.empty((BH,), np.int64))


def sparsepr_plan_export(plan: Plan) -> dict:
    """Copies the plan to host numpy arrays (synchronises)."""
    arrs = _host_arrays(plan)
    ph = PlanHost(**{k: v.ctypes.data for k, v in arrs.items()})
    _check(lib().sparsepr_plan_export(plan.handle, C.byref(ph)), "sparsepr_plan_export")
    if plan.M == 0:
        arrs["probe_idx"] = arrs["probe_idx"][:, :0]
        arrs["probe_w"] = arrs["probe_w"][:, :0]
    return arrs


def sparsepr_plan_export_features(plan: Plan, fields=("F_K", "F_Q", "phi_Q", "kappa", "theta", "score")) -> dict:
    """Copies the plan's floating-point intermediates (feature maps, query responses, group means,
    cell scores) to host numpy arrays (synchronises)."""
    BH, N, d = plan.BH, plan.shape.N, plan.shape.d
    Ck, Cq = plan.groups
    rK, rQ = min(plan.params.rK or 48, d), min(plan.params.rQ or 64, d)
    if plan.params.partition != 0:                  # semantic query partition: phi_Q holds the raw queries
        rQ = d
        fields = tuple(f for f in fields if f != "F_Q" and not (f == "F_K" and plan.params.partition == 2))
    BHkv = plan.BHkv
    shapes = dict(F_K=(BHkv, d, rK), F_Q=(BHkv, d, rQ), phi_Q=(BH, N, rQ), kappa=(BHkv, Ck, d), theta=(BH, Cq, d),
                  score=(BH, Cq, Ck))
    arrs = {k: np.empty(shapes[k], np.float32) for k in fields}
    pf = PlanFeatures(**{k: v.ctypes.data for k, v in arrs.items()})
    _check(lib().sparsepr_plan_export_features(plan.handle, C.byref(pf)), "sparsepr_plan_export_features")
    return arrs


def sparsepr_plan_import(Q, K, V, host: dict, params: Params | None = None, **kw) -> Plan:
    """Builds a device plan from host assignments, routes and probes.

    host: kv_assign/q_assign [BH,N]; route_ptr [BH,Cq+1]; route_idx [BH,Cq*Ck] slab
    (or a list of per-head index arrays); probe_idx/probe_w [BH,M]."""
    params = params or make_params(**kw)
    shape = make_shape(Q, K, V, Q)
    L = lib()
    BH, N = shape.B * shape.H, shape.N
    blk = params.block or 128
    Ck, Cq = params.Ck or -(-N // blk), params.Cq or -(-N // blk)
    a = {k: np.ascontiguousarray(host[k], dtype=np.int32) for k in ("kv_assign", "q_assign", "route_ptr")}
    ridx = host["route_idx"]
    if isinstance(ridx, (list, tuple)):
        slab = np.zeros((BH, Cq * Ck), np.int32)
        for i, r in enumerate(ridx):
            slab[i, :len(r)] = r
        ridx = slab
    a["route_idx"] = np.ascontiguousarray(ridx, dtype=np.int32)
    assert a["route_idx"].shape == (BH, Cq * Ck) and a["kv_assign"].shape == (shape.B * (shape.Hkv or shape.H), N)
    M = 0 if params.mode == 1 else min(params.n_probe, N)
    if M:
        a["probe_idx"] = np.ascontiguousarray(host["probe_idx"], dtype=np.int32)
        a["probe_w"] = np.ascontiguousarray(host["probe_w"], dtype=np.float32)
        assert a["probe_idx"].shape == (BH, M)
    ph = PlanHost(**{k: v.ctypes.data for k, v in a.items()})
    ws = _workspace(L.sparsepr_plan_workspace_bytes(C.byref(shape), C.byref(params)), Q.device)
    handle = C.c_void_p()
    _check(L.sparsepr_plan_import(C.byref(shape), C.byref(params), C.byref(ph), ws.data_ptr(), ws.numel(),
                                  _stream(), C.byref(handle)), "sparsepr_plan_import")
    return Plan(handle, ws, shape, params, L.sparsepr_attend_workspace_bytes(C.byref(shape), C.byref(params)))


def sparsepr_selftest_bounded_wait() -> int:
    """Runs one bounded device wait into its limit (harmless form) and returns the status it recorded."""
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(lib().sparsepr_selftest_bounded_wait(word.data_ptr(), _stream()), "sparsepr_selftest_bounded_wait")
    return int(word.item())


# ---- single stages -------------------------------------------------------------------
def sparsepr_stage_assign(X: torch.Tensor, mu: torch.Tensor) -> torch.Tensor:
    X, mu = X.contiguous().float(), mu.contiguous().float()
    n, r = X.shape
    Cn = mu.shape[0]
    L = lib()
    ws = _workspace(L.sparsepr_stage_assign_workspace_bytes(n, Cn, r), X.device)
    a = torch.empty(n, dtype=torch.int32, device=X.device)
    _check(L.sparsepr_stage_assign(n, Cn, r, X.data_ptr(), mu.data_ptr(), a.data_ptr(), ws.data_ptr(), ws.numel(),
                                   _stream()), "sparsepr_stage_assign")
    return a


def sparsepr_stage_assign_static(X: torch.Tensor, mu: torch.Tensor, out: torch.Tensor) -> torch.Tensor:
    """The assignment stage without any workspace: for callers that cannot allocate device
    memory (all of it already belongs to their own pool, or an allocation's device-wide
    synchronisation is not acceptable where they run).  X [n,r] and mu [C,r] must be
    contiguous float32 CUDA tensors and `out` a contiguous int32 CUDA tensor [n]; nothing
    is allocated here or in the library.  Limits n <= 16384, C <= 1024, r <= 64; calls that
    may overlap on the GPU must be serialised by the caller (they share one scratch array)."""
    for t in (X, mu):
        if t.dtype != torch.float32 or not t.is_contiguous() or not t.is_cuda:
            raise ValueError("X and mu must be contiguous float32 CUDA tensors")
    if out.dtype != torch.int32 or not out.is_contiguous() or out.numel() != X.shape[0]:
        raise ValueError("out must be a contiguous int32 tensor with one entry per row of X")
    _check(lib().sparsepr_stage_assign_static(X.shape[0], mu.shape[0], X.shape[1], X.data_ptr(), mu.data_ptr(),
                                              out.data_ptr(), _stream()), "sparsepr_stage_assign_static")
    return out


def sparsepr_stage_permute(a: torch.Tensor, Cn: int):
    a = a.contiguous().to(torch.int32)
    n = a.numel()
    perm, inv = torch.empty_like(a), torch.empty_like(a)
    off = torch.empty(Cn + 1, dtype=torch.int32, device=a.device)
    _check(lib().sparsepr_stage_permute(n, Cn, a.data_ptr(), perm.data_ptr(), inv.data_ptr(), off.data_ptr(),
                                        _stream()), "sparsepr_stage_permute")
    return perm, inv, off


def sparsepr_stage_route(score: torch.Tensor, nq: torch.Tensor, nk: torch.Tensor, budget: int, select_all=False):
    score = score.contiguous().float()
    Cq, Ck = score.shape
    nq, nk = nq.contiguous().to(torch.int32), nk.contiguous().to(torch.int32)
    ptr = torch.empty(Cq + 1, dtype=torch.int32, device=score.device)
    idx = torch.zeros(Cq * Ck, dtype=torch.int32, device=score.device)
    pairs = torch.zeros(1, dtype=torch.int64, device=score.device)
    _check(lib().sparsepr_stage_route(Cq, Ck, score.data_ptr(), nq.data_ptr(), nk.data_ptr(), int(budget),
                                      int(bool(select_all)), ptr.data_ptr(), idx.data_ptr(), pairs.data_ptr(),
                                      _stream()), "sparsepr_stage_route")
    return ptr, idx, pairs


# ---- whole call on host buffers ----------------------------------------------------------
def head_groups(B: int, H: int, Hkv: int, groups: int):
    """The groups of heads the host-buffer call pipelines: boxes (b0, b1, h0, h1)."""
    n = lib().sparsepr_head_groups(B, H, Hkv, groups, None, 0)
    buf = (C.c_int32 * (4 * max(n, 1)))()
    lib().sparsepr_head_groups(B, H, Hkv, groups, buf, n)
    return [tuple(buf[4 * i:4 * i + 4]) for i in range(n)]


def call_host_workspace(Qh, Kh, params: Params, groups=4) -> torch.Tensor:
    """Device workspace of sparsepr_call_host for tensors of these shapes (reusable between calls)."""
    shape = _host_shape(Qh, Kh)
    nbytes = lib().sparsepr_call_host_workspace_bytes(C.byref(shape), C.byref(params), groups)
    if nbytes == 0:
        raise SparsePRError(1, "sparsepr_call_host_workspace_bytes")
    return _workspace(nbytes, torch.device("cuda"))


def _host_shape(Qh, Kh) -> Shape:
    B, H, N, d = Qh.shape
    return Shape(B=B, H=H, N=N, d=d, dv=d, dtype=_dtype_code(Qh), Hkv=Kh.shape[1])


def sparsepr_call_host(Qh, Kh, Vh, Oh, params: Params, workspace=None, groups=4):
    """One full call for a user whose tensors live in (pinned) host memory: host->device copies, plan, attend,
    device->host copy of O, pipelined over `groups` groups of heads inside the library.  Returns O on host (complete
    when the call returns).  `workspace`: a tensor from call_host_workspace, allocated here if absent."""
    for t in (Qh, Kh, Vh, Oh):
        if t.is_cuda or not t.is_contiguous() or t.dim() != 4:
            raise ValueError("expected contiguous host tensors [B, H, N, d]")
    if Kh.shape != Vh.shape or Oh.shape != Qh.shape or Qh.shape[1] % Kh.shape[1] != 0:
        raise ValueError("K and V need the same shape, O the shape of Q, and H a multiple of the K/V heads")
    ws = workspace if workspace is not None else call_host_workspace(Qh, Kh, params, groups)
    shape = _host_shape(Qh, Kh)
    _check(lib().sparsepr_call_host(C.byref(shape), C.byref(params), Qh.data_ptr(), Kh.data_ptr(), Vh.data_ptr(),
                                    Oh.data_ptr(), groups, ws.data_ptr(), ws.numel(), _stream()), "sparsepr_call_host")
    return Oh
