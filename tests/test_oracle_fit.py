"""Pins for Probe-Fitted Residual Reconstruction in the oracle (Section 4.2, Appendix A.3)."""
import numpy as np

from oracle import sparsepr_oracle as orc


def _probes(rng, M=40, dv=6):
    X = rng.normal(size=(M, dv)) * rng.uniform(0.5, 3, size=dv) + rng.normal(size=dv)
    R = rng.normal(size=(M, dv))
    w = rng.uniform(0.5, 4, size=M)
    return X, R, w


def test_weight_normalisations_and_centering():
    rng = np.random.default_rng(0)
    X, R, w = _probes(rng)
    f = orc.probe_fit(X, R, w)
    assert abs(f["alpha"].sum() - 1) < 1e-14 and abs(f["wt"].sum() - 40) < 1e-12
    assert np.allclose(f["alpha"] @ f["Xb"], 0, atol=1e-13) and np.allclose(f["alpha"] @ f["Rb"], 0, atol=1e-13)
    assert np.allclose(f["alpha"] @ f["Xb"] ** 2, 1 - 1e-6 / f["s_x"] ** 2, atol=1e-12)   # unit weighted variance up to eps


def test_ridge_normal_equations_and_lstsq():
    rng = np.random.default_rng(1)
    X, R, w = _probes(rng)
    lam = 0.1
    f = orc.probe_fit(X, R, w, lam=lam, r_out=6)
    Xb, Rb, W = f["Xb"], f["Rb"], np.diag(f["wt"])
    assert np.allclose((Xb.T @ W @ Xb + lam * np.eye(6)) @ f["B"], Xb.T @ W @ Rb, atol=1e-11)
    # minimiser of ||W^(1/2)(Rb - Xb B)||^2 + lam ||B||^2 == least squares on the augmented system
    Aaug = np.concatenate([np.sqrt(f["wt"])[:, None] * Xb, np.sqrt(lam) * np.eye(6)])
    baug = np.concatenate([np.sqrt(f["wt"])[:, None] * Rb, np.zeros((6, 6))])
    assert np.allclose(np.linalg.lstsq(Aaug, baug, rcond=None)[0], f["B"], atol=1e-11)
    big = orc.probe_fit(X, R, w, lam=1e12)
    assert np.abs(big["B"]).max() < 1e-9                              # lam -> inf: B -> 0


def test_subspace_properties():
    rng = np.random.default_rng(2)
    X, R, w = _probes(rng)
    f = orc.probe_fit(X, R, w, r_out=3)
    Psi = f["Psi"]
    assert Psi.shape == (6, 3) and np.allclose(Psi.T @ Psi, np.eye(3), atol=1e-13)
    P = Psi @ Psi.T
    assert np.allclose(P @ P, P, atol=1e-13) and np.allclose(P, P.T)
    # leading eigenvectors of Rb^T W Rb span the same space
    S = f["Rb"].T @ (f["wt"][:, None] * f["Rb"])
    lam, U = np.linalg.eigh(S)
    assert np.allclose(U[:, -3:] @ U[:, -3:].T, P, atol=1e-10)
    full = orc.probe_fit(X, R, w, r_out=6)
    assert np.allclose(full["Psi"] @ full["Psi"].T, np.eye(6), atol=1e-12)   # r = d_v: identity
    few = orc.probe_fit(X[:4], R[:4], w[:4], r_out=16)
    assert few["r"] == 4


def test_zero_residual_gives_identity():
    rng = np.random.default_rng(3)
    X, _, w = _probes(rng)
    f = orc.probe_fit(X, np.zeros_like(X), w)
    Osp = rng.normal(size=(10, 6))
    assert np.all(orc.predict_residual(Osp, f) == 0)
    Oh = orc.reconstruct(Osp, [2, 5], Osp[[2, 5]] + 1.0, f)
    mask = np.ones(10, bool); mask[[2, 5]] = False
    assert np.array_equal(Oh[mask], Osp[mask]) and np.array_equal(Oh[[2, 5]], Osp[[2, 5]] + 1.0)


def test_truly_affine_residual_is_fitted_exactly():
    """R = b + x B* with rank(B*) <= r, lam = 0 and M >= d_v + 1: exact recovery on unseen rows."""
    rng = np.random.default_rng(4)
    dv, M, r = 6, 30, 2
    Bstar = rng.normal(size=(dv, r)) @ rng.normal(size=(r, dv))
    b = rng.normal(size=dv)
    X = rng.normal(size=(M, dv))
    w = rng.uniform(1, 3, size=M)
    f = orc.probe_fit(X, b + X @ Bstar, w, lam=0.0, r_out=r, eps_std=0.0)
    Xnew = rng.normal(size=(50, dv))
    assert np.allclose(orc.predict_residual(Xnew, f), b + Xnew @ Bstar, atol=1e-11)
    # the composed map (A, c) is the same prediction
    assert np.allclose(f["c"] + Xnew @ f["A"], orc.predict_residual(Xnew, f), atol=1e-12)
    # with the paper's lam = 0.1 the fit is regularised, hence not exact
    g = orc.probe_fit(X, b + X @ Bstar, w, lam=0.1, r_out=r)
    assert not np.allclose(orc.predict_residual(Xnew, g), b + Xnew @ Bstar, atol=1e-6)


def test_composed_map_equals_stepwise_prediction():
    rng = np.random.default_rng(5)
    X, R, w = _probes(rng)
    f = orc.probe_fit(X, R, w, r_out=3)
    Xn = rng.normal(size=(9, 6))
    step = f["mu_R"] + ((Xn - f["mu_x"]) / f["s_x"]) @ f["B"] @ f["Psi"] @ f["Psi"].T
    assert np.allclose(orc.predict_residual(Xn, f), step, atol=1e-14)
    assert np.allclose(f["c"] + Xn @ f["A"], step, atol=1e-12)


def test_full_call_on_small_input():
    """End to end on a small head: density accounting, probe rows exact, repair
    not worse than hard drop on the probes' own distribution, 100 % density = dense."""
    from paper_2608_18484_b200 import workloads as W
    wl = W.TINY.scaled(grid=(1, 32, 32))
    Q, K, V = W.make_head(wl, 0)
    prm = orc.default_params(density=0.25, block=64, n_sample=64, n_probe=32, softmax_scale=1.0)
    O_hat, O_sp, plan, fit = orc.sparsepr_head(Q, K, V, prm, 0)
    O = orc.dense_attention(Q, K, V, 1.0)
    assert np.allclose(O_hat[plan["probe_idx"]], O[plan["probe_idx"]], atol=1e-13)
    assert abs(plan["rho_exec"] - plan["rho_route"] - 32 / wl.N) < 1e-15
    assert plan["rho_exec"] <= 0.25 + 1e-12 or plan["routed_pairs"] > plan["budget"]
    assert 0.15 < plan["rho_exec"]
    assert orc.rel_l2(O_hat, O) < orc.rel_l2(O_sp, O)
    full = orc.default_params(density=1.0, block=64, n_sample=64, n_probe=32, softmax_scale=1.0)
    O_hat1, O_sp1, plan1, _ = orc.sparsepr_head(Q, K, V, full, 0)
    assert np.allclose(O_sp1, O, atol=1e-13) and np.allclose(O_hat1, O, atol=1e-9)
    assert plan1["rho_route"] == 1.0
    hard = orc.default_params(density=0.25, block=64, n_sample=64, n_probe=32, softmax_scale=1.0, mode=1)
    O_h, O_s, plan_h, fit_h = orc.sparsepr_head(Q, K, V, hard, 0)
    assert fit_h is None and np.array_equal(O_h, O_s) and plan_h["M"] == 0
