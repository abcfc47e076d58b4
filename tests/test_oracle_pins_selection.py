"""Pins of the oracle's dictionary selection search (Section III-A: Eq. 5-9, Algorithm 1) against things other than
itself: the Gram statistics against per-atom responses built from the already pinned dense regression, the LASSO
(Eq. 7) against a library solver, its optimality conditions and its closed forms, the re-fit (Eq. 9) against a library
least-squares solve, and the whole search against a problem whose answer is known in closed form (orthogonal
features) and against the stopping rules the algorithm states."""
import numpy as np
import pytest
from sklearn.linear_model import Lasso

import oracle
import sr_inputs


def _problem(D=10, k=3, r=2, h=9, w=11, dt="f16", seed=3, c=3):
    wl = sr_inputs.Workload("t", 2, c, h, w, r, D=D, k=k, coef_dtype=dt)
    lr, d, coef = sr_inputs.make_inputs(wl, seed=sr_inputs.BASE_SEED + seed)
    rng = np.random.default_rng(seed)
    d = (d + rng.normal(0, 0.1, d.shape)).astype(np.float32)          # asymmetric, signed atoms
    target = (oracle.dict_regress_dense(lr, coef, d, r, k) + rng.normal(0, 0.01, (2, c, h * r, w * r))).astype(np.float32)
    return wl, lr, d, coef, target


def _features(wl, lr, d, coef):
    """Z [rows = (frame, channel, Y, X)][atom]: response of every atom alone, through the pinned dense regression."""
    cols = []
    for l in range(wl.D):
        one = np.zeros_like(d)
        one[l] = d[l]
        cols.append(oracle.dict_regress_dense(lr, coef, one, wl.scale, wl.k).ravel())
    return np.stack(cols, axis=1)


@pytest.mark.parametrize("dt,k,r", [("f16", 3, 2), ("f32", 5, 3), ("f16", 1, 4)])
def test_gram_statistics_match_per_atom_responses(dt, k, r):
    wl, lr, d, coef, target = _problem(D=7, k=k, r=r, dt=dt)
    if k == 1:
        d = np.random.default_rng(0).uniform(-1, 1, (7, 1)).astype(np.float32)
        target = oracle.dict_regress_dense(lr, coef, d, r, k).astype(np.float32)
    Z = _features(wl, lr, d, coef)
    hvec = target.astype(np.float64).ravel()
    G, b, hh = oracle.selection_gram(lr, coef, d, target, None, r, k)
    scale = np.abs(Z.T @ Z).max()
    assert np.abs(G - Z.T @ Z).max() <= 1e-12 * scale
    assert np.abs(b - Z.T @ hvec).max() <= 1e-12 * scale
    assert abs(hh - hvec @ hvec) <= 1e-12 * hh
    # a sample of pixels (with a repeated one): only those rows, every channel of each
    samples = np.array([0, 5, 5, wl.H * wl.W - 1, wl.H * wl.W + 3, 2 * wl.H * wl.W - 1], dtype=np.int64)
    Zr = Z.reshape(wl.n, wl.c, wl.H * wl.W, wl.D)
    hr = hvec.reshape(wl.n, wl.c, wl.H * wl.W)
    rows = np.concatenate([Zr[s // (wl.H * wl.W), :, s % (wl.H * wl.W)] for s in samples])
    hs = np.concatenate([hr[s // (wl.H * wl.W), :, s % (wl.H * wl.W)] for s in samples])
    G, b, hh = oracle.selection_gram(lr, coef, d, target, samples, r, k)
    assert np.abs(G - rows.T @ rows).max() <= 1e-12 * max(1.0, np.abs(rows.T @ rows).max())
    assert np.abs(b - rows.T @ hs).max() <= 1e-12 * max(1.0, np.abs(rows.T @ hs).max())
    assert abs(hh - hs @ hs) <= 1e-12 * max(1.0, hh)


def _kkt(G, b, beta, n, lam):
    grad = (2.0 / n) * (b - G @ beta)                        # minus the gradient of the smooth part
    on = beta != 0
    return (np.abs(grad[on] - lam * np.sign(beta[on])).max() if on.any() else 0.0,
            (np.abs(grad[~on]) - lam).max() if (~on).any() else -np.inf)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_lasso_matches_a_library_solver_and_its_optimality_conditions(seed):
    rng = np.random.default_rng(seed)
    n, L = 400, 12
    Z = rng.normal(size=(n, L)) @ (np.eye(L) + 0.2 * rng.normal(size=(L, L)))      # correlated columns
    h = Z @ (rng.normal(size=L) * (rng.random(L) < 0.6)) + rng.normal(0, 0.3, n)
    G, b = Z.T @ Z, Z.T @ h
    for lam in (1e-3, 0.05, 0.3, 1.0, 3.0):
        beta, sweeps = oracle.lasso_cd(G, b, n, lam, max_sweeps=200000)
        assert sweeps < 200000                               # converged: the last sweep moved nothing by more than tol
        ref = Lasso(alpha=lam / 2, fit_intercept=False, tol=1e-14, max_iter=200000).fit(Z, h).coef_
        assert np.abs(beta - ref).max() <= 1e-7
        np.testing.assert_array_equal(beta != 0, ref != 0)
        on_err, off_slack = _kkt(G, b, beta, n, lam)
        assert on_err <= 1e-9 and off_slack <= 1e-9
    # lambda = 0 is least squares; lambda >= (2/N) max |b| keeps nothing
    beta, _ = oracle.lasso_cd(G, b, n, 0.0, tol=1e-14, max_sweeps=100000)
    assert np.abs(beta - np.linalg.lstsq(Z, h, rcond=None)[0]).max() <= 1e-8
    beta, _ = oracle.lasso_cd(G, b, n, 2.0 / n * np.abs(b).max() * (1 + 1e-12))
    assert not beta.any()
    # the active mask: inactive atoms stay at zero and the rest solve the reduced problem
    act = np.ones(L, np.uint8)
    act[[1, 4]] = 0
    beta, _ = oracle.lasso_cd(G, b, n, 0.05, active=act)
    keep = act.astype(bool)
    ref = Lasso(alpha=0.025, fit_intercept=False, tol=1e-14, max_iter=200000).fit(Z[:, keep], h).coef_
    assert not beta[~keep].any() and np.abs(beta[keep] - ref).max() <= 1e-7


def test_lasso_closed_form_on_orthogonal_features_and_beta_one_at_alpha_one():
    rng = np.random.default_rng(5)
    n, L = 64, 8
    Q, _ = np.linalg.qr(rng.normal(size=(n, L)))
    Z = Q * np.linspace(1.0, 2.0, L)                         # orthogonal columns of different norms
    h = Z @ np.ones(L)                                       # the full model reproduces the target: beta = 1
    G, b = Z.T @ Z, Z.T @ h
    beta, _ = oracle.lasso_cd(G, b, n, 1e-12)
    assert np.abs(beta - 1).max() <= 1e-9
    lam = 0.02
    beta, sweeps = oracle.lasso_cd(G, b, n, lam)
    want = np.sign(b) * np.maximum(np.abs(b) - lam * n / 2, 0) / np.diag(G)       # soft threshold, coordinate by coordinate
    assert np.abs(beta - want).max() <= 1e-12 and sweeps <= 3


def test_refit_is_least_squares_on_the_support():
    wl, lr, d, coef, target = _problem(D=9, k=3)
    Z = _features(wl, lr, d, coef)
    hvec = target.astype(np.float64).ravel()
    G, b, hh = oracle.selection_gram(lr, coef, d, target, None, wl.scale, wl.k)
    n = Z.shape[0]
    # one step from 9 atoms to at most 4: alpha = delta = ... the search's gamma must be the least-squares fit on its support
    idx, gamma, trace = oracle.selection_search(G, b, hh, n, 4 / 9, 5 / 9, 0.0, 1e-8)
    assert 1 <= idx.size <= 4 and trace.shape[0] == 1
    ref = np.linalg.lstsq(Z[:, idx], hvec, rcond=None)[0]
    assert np.abs(gamma - ref).max() <= 1e-8 * max(1.0, np.abs(ref).max())
    resid = hvec - Z[:, idx] @ gamma
    assert np.abs(Z[:, idx].T @ resid).max() <= 1e-8 * np.abs(b).max()             # normal equations
    assert abs(trace[0, 4] - resid @ resid / n) <= 1e-10 * max(1.0, trace[0, 4])   # the reported loss is that fit's


def test_search_on_orthogonal_features_has_a_closed_form():
    """With orthogonal features the LASSO decouples: atom l survives lambda iff |b_l| > lambda N / 2, so a step drops
    the atoms with the smallest |b_l| until floor(alpha_t L) are left. The re-fit gives gamma_l = b_l / G_ll; it is
    folded into the layer, so from the second step on the features are gamma_l z_l and the ranking quantity becomes
    |gamma_l b_l| = b_l^2 / G_ll (the energy an atom contributes). The final re-weights are b_l / G_ll whatever
    happened in the steps before."""
    rng = np.random.default_rng(9)
    n, L = 256, 16
    Q, _ = np.linalg.qr(rng.normal(size=(n, L)))
    Z = Q * rng.uniform(0.5, 2.0, L)
    truth = rng.permutation(np.linspace(0.2, 3.0, L)) * rng.choice([-1, 1], L)
    h = Z @ truth + 0.01 * rng.normal(size=n)
    G, b, hh = Z.T @ Z, Z.T @ h, h @ h
    for alpha, dalpha in ((0.25, 0.25), (0.25, 0.125), (0.5, 0.1), (0.1, 0.3)):
        idx, gamma, trace = oracle.selection_search(G, b, hh, n, alpha, dalpha, 0.0, 1e-6)
        alive, a_t, first = np.arange(L), 1.0, True
        while a_t > alpha:
            a_t = max(alpha, a_t - dalpha)
            rank = np.abs(b[alive]) if first else b[alive] ** 2 / np.diag(G)[alive]
            alive = np.sort(alive[np.argsort(-rank)[: int(np.floor(a_t * L + 1e-9))]])
            first = False
        want = alive
        np.testing.assert_array_equal(idx, want)
        assert np.abs(gamma - (b / np.diag(G))[want]).max() <= 1e-9
        # the alpha schedule: 1 - dalpha, 1 - 2 dalpha, ..., never below alpha
        steps = trace.shape[0]
        assert steps == int(np.ceil((1 - alpha) / dalpha - 1e-9))
        np.testing.assert_allclose(trace[:, 0], np.maximum(alpha, 1 - dalpha * np.arange(1, steps + 1)), atol=1e-12)


def test_search_obeys_its_stopping_rules_on_a_correlated_problem():
    wl, lr, d, coef, target = _problem(D=24, k=3, h=12, w=12)
    G, b, hh = oracle.selection_gram(lr, coef, d, target, None, wl.scale, wl.k)
    n = wl.npix * wl.c
    L, alpha, dalpha, eps = 24, 0.25, 0.125, 0.05
    idx, gamma, trace = oracle.selection_search(G, b, hh, n, alpha, dalpha, eps, 1e-9)
    assert idx.size <= alpha * L and idx.size >= 1 and np.all(np.diff(idx.astype(int)) > 0)
    kept = trace[:, 2]
    assert np.all(kept <= trace[:, 0] * L + 1e-9)                                  # || beta ||_0 <= alpha_t L at every step
    assert np.all(np.diff(kept) <= 0)                                              # atoms are only ever discarded
    assert np.all(trace[:, 4] <= trace[:, 3] + 1e-12)                              # the re-fit never raises the loss
    assert np.all(np.diff(trace[:, 1]) >= 0)                                       # lambda is carried forward and only grows
    # the final loss is that of the least-squares fit on the final support
    Z = _features(wl, lr, d, coef)
    hvec = target.astype(np.float64).ravel()
    ref = np.linalg.lstsq(Z[:, idx], hvec, rcond=None)[0]
    assert np.abs(gamma - ref).max() <= 1e-6 * max(1.0, np.abs(ref).max())


def test_search_finds_planted_atoms():
    """A stand-in for a trained model whose coefficient layer uses a few atoms much more than the rest (the paper's
    premise that the backbone extracts sparse information for the dictionary): the search keeps exactly those."""
    wl = sr_inputs.Workload("t", 1, 3, 12, 12, 2, D=16, k=3, coef_dtype="f16")
    lr, d, coef = sr_inputs.make_inputs(wl)
    important = np.array([2, 7, 11, 13])
    scale = np.full(16, 0.02, np.float32)
    scale[important] = 1.0
    coef = (coef.astype(np.float32) * scale[None, :, None, None]).astype(np.float16)
    target = oracle.dict_regress_dense(lr, coef, d, 2, 3).astype(np.float32)
    G, b, hh = oracle.selection_gram(lr, coef, d, target, None, 2, 3)
    idx, gamma, trace = oracle.selection_search(G, b, hh, wl.npix * 3, 0.25, 0.25, 0.0, 1e-9)
    np.testing.assert_array_equal(idx, important)
    full = float(hh) / (wl.npix * 3)
    assert trace[-1, 4] <= 1e-3 * full                                             # almost all of the energy is kept


def test_selection_argument_errors():
    G, b = np.eye(3), np.ones(3)
    with pytest.raises(ValueError):
        oracle.selection_search(G, b, 1.0, 10, 1.5, 0.1, 0.0, 1e-3)                # alpha > 1
    with pytest.raises(ValueError):
        oracle.selection_search(G, b, 1.0, 10, 0.5, 0.0, 0.0, 1e-3)                # no progress per step
    with pytest.raises(ValueError):
        oracle.lasso_cd(G, b, 0.0, 0.1)                                            # no rows
