"""Pins for the oracle's attention operators (Eq. 1, Eq. 3, Appendix A.1)."""
import math

import numpy as np

from oracle import sparsepr_oracle as orc


def brute_attention(Q, K, V, scale):
    """Eq. 1 by explicit Python loops and math.exp (tiny inputs only)."""
    out = []
    for q in Q:
        logits = [scale * sum(float(a) * float(b) for a, b in zip(q, k)) for k in K]
        m = max(logits)
        e = [math.exp(l - m) for l in logits]
        z = sum(e)
        out.append([sum(e[j] * float(V[j][c]) for j in range(len(K))) / z for c in range(len(V[0]))])
    return np.array(out)


def test_dense_matches_brute_force():
    rng = np.random.default_rng(1)
    Q, K, V = rng.normal(size=(7, 5)), rng.normal(size=(9, 5)), rng.normal(size=(9, 3))
    s = 1 / math.sqrt(5)
    assert np.allclose(orc.dense_attention(Q, K, V, s), brute_attention(Q, K, V, s), atol=1e-13)
    # row subset and chunking do not change values
    assert np.allclose(orc.dense_attention(Q, K, V, s, rows=[4, 1]), brute_attention(Q[[4, 1]], K, V, s), atol=1e-13)
    assert np.allclose(orc.dense_attention(Q, K, V, s, chunk=2), brute_attention(Q, K, V, s), atol=1e-13)


def test_dense_special_cases():
    rng = np.random.default_rng(2)
    Q, K = rng.normal(size=(6, 4)), rng.normal(size=(11, 4))
    V = np.tile(rng.normal(size=(1, 3)), (11, 1))
    assert np.allclose(orc.dense_attention(Q, K, V, 0.5), V[:6], atol=1e-14)       # constant V
    V = rng.normal(size=(11, 3))
    Ksame = np.tile(K[:1], (11, 1))
    assert np.allclose(orc.dense_attention(Q, Ksame, V, 0.5), np.tile(V.mean(0), (6, 1)), atol=1e-14)
    p = rng.permutation(11)                                                       # joint (K,V) permutation
    assert np.allclose(orc.dense_attention(Q, K, V, 0.5), orc.dense_attention(Q, K[p], V[p], 0.5), atol=1e-14)
    # a transposed operand or a wrong scale must show
    assert not np.allclose(orc.dense_attention(Q, K, V, 0.5), orc.dense_attention(Q, K, V, 0.25))


def _toy_partition(rng, N, Cq, Ck):
    a_Q = rng.integers(0, Cq, size=N)
    a_K = rng.integers(0, Ck, size=N)
    z = rng.random((Cq, Ck)) < 0.4
    z[np.arange(Cq), rng.integers(0, Ck, size=Cq)] = True
    ptr = np.zeros(Cq + 1, dtype=np.int32)
    ptr[1:] = np.cumsum(z.sum(1))
    idx = np.nonzero(z)[1].astype(np.int32)
    return a_Q, a_K, z, ptr, idx


def test_hard_drop_is_renormalised_softmax_over_support():
    rng = np.random.default_rng(3)
    N, d = 40, 6
    Q, K, V = rng.normal(size=(N, d)), rng.normal(size=(N, d)), rng.normal(size=(N, 4))
    a_Q, a_K, z, ptr, idx = _toy_partition(rng, N, 5, 6)
    O = orc.sparse_attention(Q, K, V, a_Q, a_K, ptr, idx, 0.4)
    for i in range(N):
        keep = z[a_Q[i], a_K]                       # key j retained iff cell (a_Q[i], a_K[j]) selected
        w = np.exp(0.4 * K @ Q[i]) * keep
        assert np.allclose(O[i], (w / w.sum()) @ V, atol=1e-13)
    # row subset agrees with the full evaluation
    assert np.allclose(orc.sparse_attention(Q, K, V, a_Q, a_K, ptr, idx, 0.4, rows=[7, 3, 30]), O[[7, 3, 30]])


def test_all_cells_reproduce_dense():
    rng = np.random.default_rng(4)
    N = 33
    Q, K, V = rng.normal(size=(N, 8)), rng.normal(size=(N, 8)), rng.normal(size=(N, 8))
    a_Q, a_K = rng.integers(0, 4, N), rng.integers(0, 3, N)
    ptr = np.arange(5, dtype=np.int32) * 3
    idx = np.tile(np.arange(3, dtype=np.int32), 4)
    assert np.allclose(orc.sparse_attention(Q, K, V, a_Q, a_K, ptr, idx, 0.3),
                       orc.dense_attention(Q, K, V, 0.3), atol=1e-14)


def test_residual_identity():
    """R_i = p_U (O_U - O_sp) and O_dense = (1 - p_U) O_sp + p_U O_U (Appendix A.1)."""
    rng = np.random.default_rng(5)
    N = 30
    Q, K, V = rng.normal(size=(N, 5)), rng.normal(size=(N, 5)), rng.normal(size=(N, 5))
    a_Q, a_K, z, ptr, idx = _toy_partition(rng, N, 4, 5)
    O_sp = orc.sparse_attention(Q, K, V, a_Q, a_K, ptr, idx, 0.7)
    O_d = orc.dense_attention(Q, K, V, 0.7)
    for i in range(N):
        keep = z[a_Q[i], a_K]
        Z_S, N_S, Z_U, N_U = orc.partition_statistics(Q[i], K, V, keep, 0.7)
        assert np.allclose(O_d[i], (N_S + N_U) / (Z_S + Z_U), atol=1e-13)
        assert np.allclose(O_sp[i], N_S / Z_S, atol=1e-13)
        if Z_U > 0:
            p_U, O_U = Z_U / (Z_S + Z_U), N_U / Z_U
            assert np.allclose(O_d[i] - O_sp[i], p_U * (O_U - O_sp[i]), atol=1e-13)
            assert np.allclose(O_d[i], (1 - p_U) * O_sp[i] + p_U * O_U, atol=1e-13)


def test_density_accounting():
    rng = np.random.default_rng(6)
    N = 50
    a_Q, a_K, z, ptr, idx = _toy_partition(rng, N, 6, 7)
    n_q, n_k = np.bincount(a_Q, minlength=6), np.bincount(a_K, minlength=7)
    brute = sum(1 for i in range(N) for j in range(N) if z[a_Q[i], a_K[j]])       # Eq. 2 by counting pairs
    pairs = orc.routed_pairs(n_q, n_k, ptr, idx)
    assert pairs == brute
    rr, re = orc.densities(pairs, N, N, 5)
    assert rr == brute / N**2 and abs(re - rr - 5 / N) < 1e-15


def test_probe_fractions_table():
    """M/N_q for M = 64 as printed in the paper's Table C.2."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "probe_fractions.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 4
    for n, pct in rows:
        _, rho_exec = orc.densities(0, int(n), int(n), 64)
        assert round(100 * rho_exec, 3) == float(pct)


def test_error_metrics():
    O = np.array([[3.0, 4.0], [0.0, 2.0]])
    Oh = np.array([[3.0, 4.0], [0.0, 1.0]])
    assert abs(orc.rel_l2(Oh, O) - 1 / math.sqrt(29)) < 1e-15
    mean, p99 = orc.row_errors(Oh, O)
    assert abs(mean - 0.25) < 1e-15
    assert orc.row_errors(Oh, O, exclude=[1]) == (0.0, 0.0)
