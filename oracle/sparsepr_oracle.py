"""fp64 CPU oracle for one SparsePR attention call.  TEST INFRASTRUCTURE ONLY.

This module restates, step by step and in the paper's notation, what one
training-free sparse self-attention call computes (Sections 3-4, Appendix A-B
of the SparsePR paper).  It exists so that the CUDA library can be checked
element by element; it is deliberately plain and slow (numpy, float64, no
blocking beyond row chunks that bound memory, no fusion, no reordering).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import it.
It shares no code with the CUDA path and imports nothing from the product
package.  All inputs are arrays handed in by the caller; the functions promote
them to float64.

Readings taken where the paper is silent (each is repeated at the function):
  * deterministic query sample / k-means init rows: an integer stride rule with
    a splitmix64 offset (`stride_sample`);
  * k-means: Lloyd iterations from data-point initial centroids, ties to the
    lowest centroid id, empty clusters keep their previous centroid; a warm
    start seeds the centroids with the current features' means over a previous
    call's partition (`kmeans`);
  * router score: centroid estimate of the per-key attention weight of a cell
    (`cell_scores`), forced arg-max cell per non-empty query group, then the
    longest prefix of the score-sorted remaining cells that fits the pair
    budget (`route_select`);
  * epsilon of the feature scale in the probe fit: 1e-6 (`probe_fit`).

Parity pins (see tests/test_oracle_*.py): every function below is pinned by a
closed form, an invariant, a brute-force evaluation or an independent library
routine EXCEPT:
  * `kmeans` (initialisation, iteration count, empty-cluster rule are this
    build's reading): parity unpinned against the paper; invariants only.
  * `cell_scores` / `route_select` (the paper defines the budget and the cost
    model but no score): parity unpinned against the paper; invariants only.
"""
from __future__ import annotations

import numpy as np

_MASK64 = (1 << 64) - 1


# --------------------------------------------------------------------------
# Deterministic sampling (Appendix B.1: "a deterministic sample of query rows")
# --------------------------------------------------------------------------
def splitmix64(x: int) -> int:
    """The standard public-domain splitmix64 output function on a 64-bit word."""
    z = (x + 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return (z ^ (z >> 31)) & _MASK64


TAG_QUERY_SAMPLE = 1
TAG_KV_INIT = 2
TAG_Q_INIT = 3


def stride_sample(n: int, N: int, seed: int, tag: int, bh: int) -> np.ndarray:
    """n distinct row indices out of N by a fixed stride with a hashed offset.

    Reading (the paper only says "deterministic sample", Appendix B.1):
    idx(s) = floor(((s*2^24 + U) * N) / (n * 2^24)), s = 0..n-1, with the 24-bit
    offset U = splitmix64(seed*0x100000001B3 + tag*0x10001 + bh) >> 40.
    For n <= N consecutive indices differ by at least one, so they are distinct.
    """
    if n > N:
        raise ValueError("cannot draw more distinct rows than there are rows")
    key = (seed * 0x100000001B3 + tag * 0x10001 + bh) & _MASK64
    U = splitmix64(key) >> 40
    out = np.empty(n, dtype=np.int64)
    for s in range(n):
        out[s] = (((s << 24) + U) * N) // (n << 24)
    return out


# --------------------------------------------------------------------------
# Dense attention (Eq. 1) and renormalised hard drop (Eq. 3)
# --------------------------------------------------------------------------
def dense_attention(Q, K, V, scale: float, rows=None, chunk: int = 2048) -> np.ndarray:
    """O = softmax(scale * Q K^T) V, Eq. 1 (scale = 1/sqrt(d) in the paper).

    `rows` restricts the evaluation to a subset of query rows (used for probe
    rows and for sampled checks at large N).  Row chunks only bound memory.
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    if rows is not None:
        Q = Q[np.asarray(rows, dtype=np.int64)]
    O = np.empty((Q.shape[0], V.shape[1]), dtype=np.float64)
    for s in range(0, Q.shape[0], chunk):
        L = scale * (Q[s:s + chunk] @ K.T)
        L -= L.max(axis=1, keepdims=True)
        P = np.exp(L)
        O[s:s + chunk] = (P @ V) / P.sum(axis=1, keepdims=True)
    return O


def sparse_attention(Q, K, V, a_Q, a_K, route_ptr, route_idx, scale: float, rows=None) -> np.ndarray:
    """Renormalised hard drop, Eq. 3: every query of group a soft-maxes over the
    keys of the K/V groups routed to a (cells with z_ab = 1) only.

    Rows of an empty support (cannot happen with `route_select`, which forces
    one cell per non-empty query group) are returned as zeros.
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    a_Q = np.asarray(a_Q)
    a_K = np.asarray(a_K)
    sel_rows = np.arange(Q.shape[0]) if rows is None else np.asarray(rows, dtype=np.int64)
    O = np.zeros((sel_rows.shape[0], V.shape[1]), dtype=np.float64)
    Cq = len(route_ptr) - 1
    for a in range(Cq):
        mine = np.nonzero(a_Q[sel_rows] == a)[0]
        if mine.size == 0:
            continue
        groups = np.asarray(route_idx[route_ptr[a]:route_ptr[a + 1]])
        keys = np.nonzero(np.isin(a_K, groups))[0]      # K_a, V_a of Eq. 3
        if keys.size == 0:
            continue
        O[mine] = dense_attention(Q[sel_rows[mine]], K[keys], V[keys], scale)
    return O


def partition_statistics(q, K, V, retained_mask, scale: float):
    """Z_S, N_S, Z_U, N_U of Appendix A.1 for one query row (un-shifted
    exponentials; use on small logits only)."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    e = np.exp(scale * (K @ q))
    S = np.asarray(retained_mask, dtype=bool)
    return e[S].sum(), e[S] @ V[S], e[~S].sum(), e[~S] @ V[~S]


# --------------------------------------------------------------------------
# Density accounting (Eq. 2; Section 4.3)
# --------------------------------------------------------------------------
def routed_pairs(n_q, n_k, route_ptr, route_idx) -> int:
    """sum_ab z_ab |G_a^Q| |G_b^KV| as an exact integer."""
    total = 0
    for a in range(len(route_ptr) - 1):
        for b in route_idx[route_ptr[a]:route_ptr[a + 1]]:
            total += int(n_q[a]) * int(n_k[b])
    return total


def densities(pairs: int, N_q: int, N_k: int, M: int):
    """rho_route (Eq. 2) and rho_exec = rho_route + M/N_q (Section 4.3)."""
    rho_route = pairs / (N_q * N_k)
    return rho_route, rho_route + M / N_q


# --------------------------------------------------------------------------
# Response coordinates (Section 4.1, Appendix B)
# --------------------------------------------------------------------------
def key_response_metric(Q_s) -> np.ndarray:
    """M_K = Q_s^T Q_s / M_s (Appendix B.1)."""
    Q_s = np.asarray(Q_s, dtype=np.float64)
    return Q_s.T @ Q_s / Q_s.shape[0]


def eig_feature_map(Mmat, r: int):
    """F = U_r diag(sqrt(lambda_i / mean_{j<=r} lambda_j)): leading r
    eigendirections scaled by the square roots of their eigenvalues after the
    retained eigenvalues are normalised to unit mean (Section 4.1).

    Negative round-off eigenvalues are clamped to 0; an all-zero retained
    spectrum gives F = 0.  Returns (F, retained eigenvalues).
    """
    Mmat = np.asarray(Mmat, dtype=np.float64)
    d = Mmat.shape[0]
    r = min(r, d)
    lam, U = np.linalg.eigh(0.5 * (Mmat + Mmat.T))
    order = np.argsort(-lam, kind="stable")
    lam = np.maximum(lam[order][:r], 0.0)
    U = U[:, order][:, :r]
    mean = lam.mean()
    if mean <= 0.0:
        return np.zeros((d, r)), lam
    return U * np.sqrt(lam / mean)[None, :], lam


def key_response(K, F_K) -> np.ndarray:
    """phi_K(k_j) = F_K^T k_j (Eq. 6)."""
    return np.asarray(K, dtype=np.float64) @ np.asarray(F_K, dtype=np.float64)


def kv_centroids(K, a_K, C_k: int):
    """Original-space centroid kappa_b of every K/V group and the group sizes
    (Appendix B.2).  Rows of empty groups are zero."""
    K = np.asarray(K, dtype=np.float64)
    a_K = np.asarray(a_K)
    n = np.bincount(a_K, minlength=C_k).astype(np.int64)
    kappa = np.zeros((C_k, K.shape[1]), dtype=np.float64)
    np.add.at(kappa, a_K, K)
    nz = n > 0
    kappa[nz] /= n[nz, None]
    return kappa, n


def query_response_metric(kappa, n_k) -> np.ndarray:
    """M_Q = Ktilde^T Ktilde / (C_k^+ d): centroids of the NON-EMPTY groups,
    centred by their uniform (not token-weighted) mean (Appendix B.2)."""
    kappa = np.asarray(kappa, dtype=np.float64)
    nz = np.asarray(n_k) > 0
    Kt = kappa[nz]
    Kt = Kt - Kt.mean(axis=0, keepdims=True)
    return Kt.T @ Kt / (Kt.shape[0] * kappa.shape[1])


def query_response(Q, F_Q, eps: float = 1e-6) -> np.ndarray:
    """phi_Q(q) = F_Q^T q / max(sqrt(||F_Q^T q||^2 / r_Q), eps) (Eq. 7); r_Q is
    the retained rank (number of columns of F_Q)."""
    Y = np.asarray(Q, dtype=np.float64) @ np.asarray(F_Q, dtype=np.float64)
    rms = np.sqrt((Y * Y).sum(axis=1) / Y.shape[1])
    return Y / np.maximum(rms, eps)[:, None]


# --------------------------------------------------------------------------
# k-means (Section 4.1: "applying k-means to phi")
# --------------------------------------------------------------------------
def kmeans_assign(X, mu, chunk: int = 1024) -> np.ndarray:
    """a[j] = argmin_c sum_k (X[j,k] - mu[c,k])^2, ties to the lowest c.

    The squared distance is accumulated in float64 over k = 0, 1, ... in that
    order (one multiply, one add per term, no fused multiply-add), so that an
    implementation that repeats the same sequence reproduces the decision
    exactly.
    """
    X = np.asarray(X, dtype=np.float64)
    mu = np.asarray(mu, dtype=np.float64)
    a = np.empty(X.shape[0], dtype=np.int32)
    for s in range(0, X.shape[0], chunk):
        Xc = X[s:s + chunk]
        D = np.zeros((Xc.shape[0], mu.shape[0]), dtype=np.float64)
        for k in range(X.shape[1]):
            diff = Xc[:, k][:, None] - mu[:, k][None, :]
            D = D + diff * diff
        a[s:s + chunk] = np.argmin(D, axis=1)       # first minimum = lowest id
    return a


def kmeans(X, C: int, init_rows, T: int, init_assign=None):
    """Lloyd's algorithm.  Reading (the paper fixes none of this): initial
    centroids are the feature rows `init_rows`; for t = 1..T assign, and if
    t < T move every non-empty cluster to the mean of its members while an
    empty cluster keeps its previous centroid.  Returns (a^(T), the centroids
    used by the last assignment).

    Warm start (Appendix C.1 only says the k-means is "warm-started"; reading):
    with `init_assign`, the partition of a previous call over the same token
    grid, the initial centroid of cluster c is the mean of the CURRENT features
    of the tokens that partition put in c; a cluster it left empty starts from
    its feature row of `init_rows`.  Seeding by assignment rather than by the
    previous centroids keeps the start independent of the sign and rotation
    gauge of the feature map, which may change between calls."""
    X = np.asarray(X, dtype=np.float64)
    mu = X[np.asarray(init_rows, dtype=np.int64)].copy()
    assert mu.shape[0] == C
    if init_assign is not None:
        a0 = np.asarray(init_assign)
        n0 = np.bincount(a0, minlength=C)
        s0 = np.zeros_like(mu)
        np.add.at(s0, a0, X)
        nz0 = n0 > 0
        mu[nz0] = s0[nz0] / n0[nz0, None]
    a = None
    for t in range(1, T + 1):
        a = kmeans_assign(X, mu)
        if t < T:
            n = np.bincount(a, minlength=C)
            s = np.zeros_like(mu)
            np.add.at(s, a, X)
            nz = n > 0
            mu = mu.copy()
            mu[nz] = s[nz] / n[nz, None]
    return a, mu


def kmeans_objective(X, mu, a) -> float:
    X = np.asarray(X, dtype=np.float64)
    return float(((X - np.asarray(mu, dtype=np.float64)[a]) ** 2).sum())


# --------------------------------------------------------------------------
# Group-major permutation (Section 4.3)
# --------------------------------------------------------------------------
def group_permutation(a, C: int):
    """Stable counting sort by group id.  perm[p] = original index of the token
    at group-major position p (group id ascending, original index ascending
    inside a group); inv[perm[p]] = p; off = ragged group offsets (C+1)."""
    a = np.asarray(a)
    perm = np.argsort(a, kind="stable").astype(np.int32)
    inv = np.empty_like(perm)
    inv[perm] = np.arange(a.shape[0], dtype=np.int32)
    off = np.zeros(C + 1, dtype=np.int32)
    off[1:] = np.cumsum(np.bincount(a, minlength=C))
    return perm, inv, off


# --------------------------------------------------------------------------
# Router (Section 4.3)
# --------------------------------------------------------------------------
def query_centroids(Q, a_Q, C_q: int):
    """theta_a: mean original-space query of each query group (zero if empty)."""
    return kv_centroids(Q, a_Q, C_q)


def cell_scores(theta, kappa, n_q, n_k, scale: float) -> np.ndarray:
    """Reading (the paper gives no score): p_ab = exp(l_ab - LSE_a) with
    l_ab = scale * theta_a . kappa_b and LSE_a = log sum_{b non-empty}
    n_b exp(l_ab), i.e. the attention weight a query at the group centroid
    would give to ONE key at the centroid of group b.  Cells of an empty row or
    column score 0.  Returned as float32: selection compares these 32-bit
    values."""
    theta = np.asarray(theta, dtype=np.float64)
    kappa = np.asarray(kappa, dtype=np.float64)
    n_q = np.asarray(n_q)
    n_k = np.asarray(n_k)
    l = scale * (theta @ kappa.T)
    colmask = n_k > 0
    lm = np.where(colmask[None, :], l, -np.inf)
    m = lm.max(axis=1, keepdims=True)
    lse = m + np.log((np.where(colmask, n_k, 0)[None, :] * np.exp(lm - m)).sum(axis=1, keepdims=True))
    p = np.exp(lm - lse)
    p[n_q == 0, :] = 0.0
    p[:, ~colmask] = 0.0
    return p.astype(np.float32)


def pair_budget(density: float, N_q: int, N_k: int, M: int) -> int:
    """P = floor(density * N_q * N_k) - M * N_k, clamped at 0: the probe rows'
    cost is reserved before any cell is selected (Section 4.3).  `density` is
    taken as the float32 value a C caller would pass."""
    total = int(np.floor(np.float64(np.float32(density)) * np.float64(N_q) * np.float64(N_k)))
    return max(total - M * N_k, 0)


def route_select(score, n_q, n_k, budget: int, select_all: bool = False):
    """Cell selection under a query-key pair budget, each cell charged
    |G_a^Q| |G_b^KV| (Section 4.3).  Reading of the unspecified parts:
      1. every non-empty query group first receives its highest-scoring
         non-empty cell (ties to the lowest b) so that no row has an empty
         support; these forced cells are kept even if they alone exceed the
         budget;
      2. the other cells with both groups non-empty are ordered by
         (score descending, a ascending, b ascending) on the float32 score
         values and the LONGEST PREFIX whose cumulative cost, on top of the
         forced cost, stays <= budget is taken (the first cell that does not
         fit ends the selection);
      3. `select_all` (a density target >= 1) takes every non-empty cell.
    Returns (route_ptr[C_q+1], route_idx ascending inside a row, routed pairs).
    """
    score = np.asarray(score, dtype=np.float32)
    n_q = np.asarray(n_q, dtype=np.int64)
    n_k = np.asarray(n_k, dtype=np.int64)
    C_q, C_k = score.shape
    z = np.zeros((C_q, C_k), dtype=bool)
    live = (n_q[:, None] > 0) & (n_k[None, :] > 0)
    if select_all:
        z = live.copy()
    else:
        spent = 0
        for a in range(C_q):
            if n_q[a] == 0 or not live[a].any():
                continue
            cand = np.where(live[a], score[a], np.float32(-1.0))
            b = int(np.argmax(cand))                  # first maximum = lowest b
            z[a, b] = True
            spent += int(n_q[a] * n_k[b])
        rest = np.nonzero(live & ~z)
        aa, bb = rest[0], rest[1]
        order = np.lexsort((bb, aa, -score[aa, bb].astype(np.float64)))
        for t in order:
            cost = int(n_q[aa[t]] * n_k[bb[t]])
            if spent + cost > budget:
                break
            spent += cost
            z[aa[t], bb[t]] = True
    route_ptr = np.zeros(C_q + 1, dtype=np.int32)
    route_ptr[1:] = np.cumsum(z.sum(axis=1))
    route_idx = np.nonzero(z)[1].astype(np.int32)
    pairs = int((z * (n_q[:, None] * n_k[None, :])).sum())
    return route_ptr, route_idx, pairs


# --------------------------------------------------------------------------
# Probe selection (Algorithm A.1) and coverage weights (Appendix A.2)
# --------------------------------------------------------------------------
def probe_select(a_Q, phi_Q, C_q: int, M: int):
    """Query-group-stratified exact probe selection, Algorithm A.1, stated as a ranking.

    Every row gets a radial rank inside its query group: its position when the
    group's rows are ordered by increasing distance d_i to the group centroid
    c_a in phi_Q space, ties by the original row index.  The round-robin
    traversal of the algorithm (round t takes the rank-t row of every group
    that still has one, groups in ascending id -- the "deterministic group
    order" is not specified further) visits the rows in the order of
    (radial rank, group id); the probe set is the first M rows of that order
    (all rows if M >= N_q).  Returns (probe indices in selection order, weights
    w_p = |G_a| / m_a with m_a the number of probes of group a, Appendix A.2).
    """
    a_Q = np.asarray(a_Q)
    phi_Q = np.asarray(phi_Q, dtype=np.float64)
    N = a_Q.shape[0]
    M = min(M, N)
    sizes = np.bincount(a_Q, minlength=C_q)
    c = np.zeros((C_q, phi_Q.shape[1]))
    np.add.at(c, a_Q, phi_Q)
    c[sizes > 0] /= sizes[sizes > 0, None]
    dist = np.sqrt(((phi_Q - c[a_Q]) ** 2).sum(axis=1))
    by_group = np.lexsort((np.arange(N), dist, a_Q))          # group id, then distance, then row index
    start = np.concatenate(([0], np.cumsum(sizes)))[:-1]
    rank = np.empty(N, dtype=np.int64)
    rank[by_group] = np.arange(N) - start[a_Q[by_group]]
    probes = np.lexsort((a_Q, rank))[:M].astype(np.int32)     # radial rank, then group id
    m_a = np.bincount(a_Q[probes], minlength=C_q)
    w = sizes[a_Q[probes]] / m_a[a_Q[probes]]
    return probes, w.astype(np.float64)


# --------------------------------------------------------------------------
# Weighted affine fit and probe-residual subspace (Appendix A.3)
# --------------------------------------------------------------------------
def probe_fit(X_P, R_P, w, lam: float = 0.1, r_out: int = 16, eps_std: float = 1e-6):
    """Fit R ~ mu_R + xbar B_lambda Psi_r Psi_r^T from the probe pairs.

    Steps, in the order of Appendix A.3: alpha_p = w_p / sum w; weighted means
    mu_x, mu_R; elementwise scale s_x = sqrt(sum alpha_p (x_p - mu_x)^2 + eps)
    (eps is not given in the paper: 1e-6 here); Xbar, Rbar; unit-mean weights
    wt_p = M w_p / sum w; B_lambda solves (Xbar^T W Xbar + lam I) B = Xbar^T W Rbar;
    Psi_r = leading r right singular vectors of W^{1/2} Rbar, r = min(r_out, M, d_v).
    Also returns the composed affine map (A, c) with Rhat_i = c + x_i A,
    A = diag(1/s_x) B_lambda Psi_r Psi_r^T and c = mu_R - mu_x A.
    """
    X_P = np.asarray(X_P, dtype=np.float64)
    R_P = np.asarray(R_P, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    M, d_v = X_P.shape
    alpha = w / w.sum()
    mu_x = alpha @ X_P
    mu_R = alpha @ R_P
    s_x = np.sqrt(alpha @ ((X_P - mu_x) ** 2) + eps_std)
    Xb = (X_P - mu_x) / s_x
    Rb = R_P - mu_R
    wt = M * w / w.sum()
    G = Xb.T @ (wt[:, None] * Xb) + lam * np.eye(d_v)
    B = np.linalg.solve(G, Xb.T @ (wt[:, None] * Rb))
    r = min(r_out, M, d_v)
    _, _, Vt = np.linalg.svd(np.sqrt(wt)[:, None] * Rb, full_matrices=True)
    Psi = Vt[:r].T
    A = (B @ Psi @ Psi.T) / s_x[:, None]
    c = mu_R - mu_x @ A
    return dict(alpha=alpha, mu_x=mu_x, mu_R=mu_R, s_x=s_x, Xb=Xb, Rb=Rb, wt=wt,
                B=B, Psi=Psi, A=A, c=c, r=r)


def predict_residual(X, fit) -> np.ndarray:
    """Rhat_i = mu_R + xbar_i B_lambda Psi_r Psi_r^T (Eq. 9), written out
    without the composed map."""
    Xb = (np.asarray(X, dtype=np.float64) - fit["mu_x"]) / fit["s_x"]
    return fit["mu_R"] + Xb @ fit["B"] @ fit["Psi"] @ fit["Psi"].T


def reconstruct(O_sp, probe_idx, O_dense_probe, fit) -> np.ndarray:
    """Ohat_i = O^dense_i for probes, O^sp_i + Rhat_i otherwise (Eq. 10)."""
    O_hat = np.asarray(O_sp, dtype=np.float64) + predict_residual(O_sp, fit)
    O_hat[np.asarray(probe_idx, dtype=np.int64)] = O_dense_probe
    return O_hat


# --------------------------------------------------------------------------
# The whole call for one head
# --------------------------------------------------------------------------
# Partition variants of the ablation (Section 5.2, Table 2; Section 3.1 for the semantic reference partition)
PARTITION_RESPONSE_COUPLED = 0   # K/V groups from key responses, query groups from query responses (the method)
PARTITION_KEY_RESPONSE_KV = 1    # only the K/V partition is response-based; queries are clustered semantically
PARTITION_SEMANTIC = 2           # k-means on the raw key and on the raw query activations, separately


def default_params(**kw):
    p = dict(density=0.25, block=128, Ck=0, Cq=0, n_sample=256, n_probe=128,
             rK=48, rQ=64, r_out=16, lam=0.1, eps_rms=1e-6, eps_std=1e-6,
             kmeans_iters=8, softmax_scale=0.0, seed=0, mode=0, partition=PARTITION_RESPONSE_COUPLED)
    p.update(kw)
    return p


def plan_head(Q, K, prm: dict, bh: int, warm=None):
    """Stages 1-2 of the call for one head: Response-Coupled Partitioning,
    permutations, probe selection and routing.  Returns a dict of every
    intermediate (so that single stages of another implementation can be fed
    from it).  `warm` = {"a_K": ..., "a_Q": ...}, the partition of a previous
    call, warm-starts both k-means runs (see `kmeans`).

    prm["partition"] selects the ablation variants: the semantic reference
    partition applies k-means to the raw key and query activations (Section
    3.1); the key-response K/V variant changes only the K/V partition (Section
    5.2).  Same initial rows, iteration count and tie rules in every variant.
    Where the query partition is semantic, the probe ranking of Algorithm A.1
    measures its distances in the raw query space, the space that partition
    was built in (reading: the paper runs the ablation with fixed probes)."""
    kv = plan_kv([Q], K, prm, bh, [bh], warm=warm)
    return plan_query(Q, kv, prm, bh, warm=warm)


def plan_kv(Qs, K, prm: dict, kv_bh: int, q_bhs, warm=None):
    """The K/V side of the plan for one K/V head and the query heads `Qs` that attend to it (one for ordinary
    multi-head attention; several under grouped-query attention, where the K/V partition and its metadata are
    shared by the associated query heads, Section 4.3).

    Reading for the grouped case (the paper does not say which query rows feed the key-response metric): every
    associated query head contributes its own deterministic sample of M_s rows (sample offset keyed by the query
    head's index) and M_K is the second moment of all of them together; the k-means initial rows are keyed by the
    K/V head's index.  With one query head this is exactly the single-head plan."""
    K = np.asarray(K, dtype=np.float64)
    Qs = [np.asarray(Q, dtype=np.float64) for Q in Qs]
    N, d = K.shape
    C_k = prm["Ck"] or -(-N // prm["block"])
    seed = prm["seed"]
    variant = prm.get("partition", PARTITION_RESPONSE_COUPLED)
    wK = None if warm is None else warm["a_K"]
    T = prm["kmeans_iters"]
    s_idx = [stride_sample(min(prm["n_sample"], N), N, seed, TAG_QUERY_SAMPLE, bh) for bh in q_bhs]
    M_K = F_K = lam_K = M_Q = F_Q = lam_Q = None
    if variant == PARTITION_SEMANTIC:
        phi_K = K                                   # k-means on the key activations themselves
    else:
        M_K = key_response_metric(np.concatenate([Q[i] for Q, i in zip(Qs, s_idx)], axis=0))
        F_K, lam_K = eig_feature_map(M_K, prm["rK"])
        phi_K = key_response(K, F_K)
    a_K, mu_K = kmeans(phi_K, C_k, stride_sample(C_k, N, seed, TAG_KV_INIT, kv_bh), T, init_assign=wK)
    kappa, n_k = kv_centroids(K, a_K, C_k)
    if variant == PARTITION_RESPONSE_COUPLED:
        M_Q = query_response_metric(kappa, n_k)
        F_Q, lam_Q = eig_feature_map(M_Q, prm["rQ"])
    kv_perm, kv_inv, kv_off = group_permutation(a_K, C_k)
    return dict(C_k=C_k, sample_idx=s_idx[0], sample_idx_all=s_idx, M_K=M_K, F_K=F_K, lam_K=lam_K, phi_K=phi_K, a_K=a_K,
                mu_K=mu_K, kappa=kappa, n_k=n_k, M_Q=M_Q, F_Q=F_Q, lam_Q=lam_Q, kv_perm=kv_perm, kv_inv=kv_inv,
                kv_off=kv_off)


def plan_query(Q, kv: dict, prm: dict, bh: int, warm=None):
    """The query side of the plan for one query head given the K/V side `kv` it attends to: query responses,
    query partition, probes, cell scores and routes.  Returns the K/V side's entries as well."""
    Q = np.asarray(Q, dtype=np.float64)
    N, d = Q.shape
    C_k = kv["C_k"]
    C_q = prm["Cq"] or -(-N // prm["block"])
    M = min(prm["n_probe"], N) if prm["mode"] == 0 else 0
    scale = prm["softmax_scale"] or 1.0 / np.sqrt(d)
    seed = prm["seed"]
    variant = prm.get("partition", PARTITION_RESPONSE_COUPLED)
    wQ = None if warm is None else warm["a_Q"]
    kappa, n_k = kv["kappa"], kv["n_k"]
    if variant == PARTITION_RESPONSE_COUPLED:
        phi_Q = query_response(Q, kv["F_Q"], prm["eps_rms"])
    else:
        phi_Q = Q                                   # k-means on the query activations themselves
    a_Q, mu_Q = kmeans(phi_Q, C_q, stride_sample(C_q, N, seed, TAG_Q_INIT, bh), prm["kmeans_iters"], init_assign=wQ)
    theta, n_q = query_centroids(Q, a_Q, C_q)
    q_perm, q_inv, q_off = group_permutation(a_Q, C_q)
    if M > 0:
        probe_idx, probe_w = probe_select(a_Q, phi_Q, C_q, M)
    else:
        probe_idx, probe_w = np.zeros(0, np.int32), np.zeros(0)
    score = cell_scores(theta, kappa, n_q, n_k, scale)
    budget = pair_budget(prm["density"], N, N, M)
    route_ptr, route_idx, pairs = route_select(score, n_q, n_k, budget,
                                               select_all=np.float32(prm["density"]) >= 1.0)
    out = dict(kv)
    out.update(C_q=C_q, M=M, scale=scale, phi_Q=phi_Q, a_Q=a_Q, mu_Q=mu_Q, theta=theta, n_q=n_q, q_perm=q_perm,
               q_inv=q_inv, q_off=q_off, probe_idx=probe_idx, probe_w=probe_w, score=score, budget=budget,
               route_ptr=route_ptr, route_idx=route_idx, routed_pairs=pairs)
    out["rho_route"], out["rho_exec"] = densities(pairs, N, N, M)
    return out


def plan_group(Qs, K, prm: dict, kv_bh: int, first_q_bh: int, warm=None):
    """Grouped-query attention: the plans of the query heads first_q_bh, first_q_bh + 1, ... that share K/V head
    kv_bh.  One K/V side, one query side per query head.  `warm` = {"a_K": ..., "a_Q": [one per query head]}."""
    bhs = [first_q_bh + g for g in range(len(Qs))]
    kv = plan_kv(Qs, K, prm, kv_bh, bhs, warm=warm)
    return [plan_query(Q, kv, prm, bh, warm=None if warm is None else dict(a_K=warm["a_K"], a_Q=warm["a_Q"][g]))
            for g, (Q, bh) in enumerate(zip(Qs, bhs))]


def attend_head(Q, K, V, plan: dict, prm: dict, rows=None):
    """Stages 3-4 for one head given a plan: block-sparse attention (Eq. 3),
    exact probe rows, the fit, and the corrected output (Eq. 10).

    With `rows` only those output rows are produced (the fit always uses the
    full probe set).  Returns (O_hat, O_sp, fit or None).
    """
    scale = plan["scale"]
    args = (plan["a_Q"], plan["a_K"], plan["route_ptr"], plan["route_idx"], scale)
    O_sp = sparse_attention(Q, K, V, *args, rows=rows)
    P = plan["probe_idx"]
    if plan["M"] == 0:
        return O_sp.copy(), O_sp, None
    X_P = sparse_attention(Q, K, V, *args, rows=P)
    O_dense_P = dense_attention(Q, K, V, scale, rows=P)
    fit = probe_fit(X_P, O_dense_P - X_P, plan["probe_w"], prm["lam"], prm["r_out"], prm["eps_std"])
    O_hat = O_sp + predict_residual(O_sp, fit)
    sel = np.arange(np.asarray(Q).shape[0]) if rows is None else np.asarray(rows, dtype=np.int64)
    pos = {int(p): t for t, p in enumerate(P)}
    for t, i in enumerate(sel):
        if int(i) in pos:
            O_hat[t] = O_dense_P[pos[int(i)]]
    return O_hat, O_sp, fit


def sparsepr_head(Q, K, V, prm: dict, bh: int = 0):
    """One full SparsePR call for one head: plan then attend."""
    plan = plan_head(Q, K, prm, bh)
    O_hat, O_sp, fit = attend_head(Q, K, V, plan, prm)
    return O_hat, O_sp, plan, fit


# --------------------------------------------------------------------------
# Error metrics
# --------------------------------------------------------------------------
def rel_l2(O_hat, O_ref) -> float:
    """||O_hat - O_ref||_F / ||O_ref||_F."""
    O_hat = np.asarray(O_hat, dtype=np.float64)
    O_ref = np.asarray(O_ref, dtype=np.float64)
    return float(np.linalg.norm(O_hat - O_ref) / np.linalg.norm(O_ref))


def row_errors(O_hat, O_ref, exclude=None):
    """Per-row ||O_hat_i - O_i|| / ||O_i|| over unprobed rows: (mean, p99).
    Reading of the "normalized attention-output error" of Tables 2-4, which the
    paper does not define."""
    O_hat = np.asarray(O_hat, dtype=np.float64)
    O_ref = np.asarray(O_ref, dtype=np.float64)
    e = np.linalg.norm(O_hat - O_ref, axis=1) / np.linalg.norm(O_ref, axis=1)
    if exclude is not None and len(exclude):
        keep = np.ones(e.shape[0], dtype=bool)
        keep[np.asarray(exclude, dtype=np.int64)] = False
        e = e[keep]
    return float(e.mean()), float(np.percentile(e, 99))
