"""The dictionary selection search (Section III-A, Algorithm 1) on the GPU against the oracle: the Gram statistics
within the fp32 bound of their 32-pixel partial sums, the search bit for bit on identical statistics (same kept atoms,
same lambda path, same losses), and the two together end to end into the global-subset regression."""
import numpy as np
import pytest
import torch

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, dev, host, signed_asymmetric_dictionary

pytestmark = pytest.mark.gpu


def _problem(D, k, r, h, w, dt="f16", n=1, c=3, seed=0, planted=None):
    wl = sr_inputs.Workload("t", n, c, h, w, r, D=D, k=k, coef_dtype=dt)
    lr, d, coef = sr_inputs.make_inputs(wl, seed=sr_inputs.BASE_SEED + seed)
    d = signed_asymmetric_dictionary(d, seed=seed) if k > 1 else np.random.default_rng(seed).uniform(-1, 1, d.shape).astype(np.float32)
    if planted is not None:                                   # a few atoms carry most of the coefficient energy
        scale = np.full(D, 0.03, np.float32)
        scale[planted] = 1.0
        coef = (coef.astype(np.float32) * scale[None, :, None, None]).astype(coef.dtype)
    rng = np.random.default_rng(seed + 1)
    target = (oracle.dict_regress_dense(lr, coef, d, r, k) + rng.normal(0, 0.01, (n, c, h * r, w * r))).astype(np.float32)
    return wl, lr, d, coef, target


def _gram_close(got, want_G, want_b, want_hh):
    G, b, hh = (host(t) for t in got)
    dg = np.sqrt(np.diag(want_G))
    assert np.all(np.abs(G - want_G) <= 2e-5 * np.outer(dg, dg) + 1e-30)
    assert np.all(np.abs(b - want_b) <= 2e-5 * dg * np.sqrt(want_hh) + 1e-30)
    assert abs(hh[0] - want_hh) <= 1e-6 * want_hh
    np.testing.assert_array_equal(G, G.T)                    # both triangles are summed from the same products


@pytest.mark.parametrize("D,k,r,h,w,dt,n,c", [(72, 5, 4, 10, 12, "f16", 1, 3), (16, 3, 2, 9, 7, "f32", 2, 3), (128, 7, 3, 6, 8, "f16", 1, 1),
                                              (7, 1, 2, 5, 5, "f16", 1, 2), (33, 5, 2, 8, 8, "f16", 1, 3)])
def test_gram_statistics_match_the_oracle(D, k, r, h, w, dt, n, c):
    wl, lr, d, coef, target = _problem(D, k, r, h, w, dt, n, c)
    want = oracle.selection_gram(lr, coef, d, target, None, r, k)
    _gram_close(sr.sr_selection_gram(dev(lr), dev(coef), dev(d), dev(target), None, r, k), *want)
    # a sample with repeats and out-of-range entries (those are skipped), not a multiple of the 32-pixel chunk
    rng = np.random.default_rng(2)
    samples = rng.integers(0, wl.npix, size=77, dtype=np.int64)
    samples[5] = samples[6]
    want = oracle.selection_gram(lr, coef, d, target, samples, r, k)
    with_bad = np.concatenate([samples, np.array([-1, wl.npix, 1 << 40], dtype=np.int64)])
    _gram_close(sr.sr_selection_gram(dev(lr), dev(coef), dev(d), dev(target), dev(with_bad), r, k), *want)
    # the bilinear form of stage 1, and twice the same call gives the same bits
    want = oracle.selection_gram(lr, coef, d, target, None, r, k, flags=oracle.UPSAMPLE_BILINEAR)
    a = sr.sr_selection_gram(dev(lr), dev(coef), dev(d), dev(target), None, r, k, sr.SR_UPSAMPLE_BILINEAR)
    _gram_close(a, *want)
    b = sr.sr_selection_gram(dev(lr), dev(coef), dev(d), dev(target), None, r, k, sr.SR_UPSAMPLE_BILINEAR)
    assert all(torch.equal(x, y) for x, y in zip(a, b))


SEARCHES = [  # D, alpha, delta_alpha, eps
    (24, 0.25, 0.125, 0.05), (16, 0.5, 0.25, 0.0), (72, 0.125, 0.125, 0.02), (40, 0.1, 0.3, 0.0), (9, 1.0 / 3, 1.0 / 3, 0.0)]


@pytest.mark.parametrize("D,alpha,dalpha,eps", SEARCHES)
def test_search_is_bit_identical_on_identical_statistics(D, alpha, dalpha, eps):
    wl, lr, d, coef, target = _problem(D, 3, 2, 10, 10, seed=D)
    G, b, hh = oracle.selection_gram(lr, coef, d, target, None, 2, 3)
    nrows = wl.npix * wl.c
    kw = dict(tol=1e-9, max_sweeps=2000, max_bisect=30)
    want_idx, want_gamma, want_trace = oracle.selection_search(G, b, hh, nrows, alpha, dalpha, eps, 1e-9, **kw)
    idx, gamma, trace = sr.sr_selection_search(dev(G), dev(b), dev(np.array([hh])), nrows, alpha, dalpha, eps, 1e-9, **kw)
    np.testing.assert_array_equal(host(idx), want_idx)
    np.testing.assert_array_equal(host(trace), want_trace)    # alpha_t, lambda, atoms kept, both losses, solves: same bits
    np.testing.assert_array_equal(host(gamma), want_gamma.astype(np.float32))


def test_search_on_orthogonal_features_and_a_singular_refit():
    rng = np.random.default_rng(4)
    n, L = 256, 16
    Q, _ = np.linalg.qr(rng.normal(size=(n, L)))
    Z = Q * rng.uniform(0.5, 2.0, L)
    h = Z @ (rng.permutation(np.linspace(0.2, 3.0, L)) * rng.choice([-1, 1], L)) + 0.01 * rng.normal(size=n)
    G, b, hh = Z.T @ Z, Z.T @ h, h @ h
    want = oracle.selection_search(G, b, hh, n, 0.25, 0.125, 0.0, 1e-6, tol=1e-9, max_sweeps=2000)
    idx, gamma, trace = sr.sr_selection_search(dev(G), dev(b), dev(np.array([hh])), n, 0.25, 0.125, 0.0, 1e-6)
    np.testing.assert_array_equal(host(idx), want[0])
    np.testing.assert_array_equal(host(trace), want[2])
    # an atom that never responds (zero row and column of G) cannot be dropped by the LASSO and makes the re-fit
    # singular: both sides report it instead of returning numbers
    G0, b0 = np.diag([1.0, 2.0, 0.0, 3.0]), np.array([1.0, 1.5, 0.0, 2.0])
    with pytest.raises(ValueError):
        oracle.selection_search(G0, b0, 5.0, 10, 0.75, 0.25, 0.0, 1e-3)
    with pytest.raises(sr.SrError):
        sr.sr_selection_search(dev(G0), dev(b0), dev(np.array([5.0])), 10, 0.75, 0.25, 0.0, 1e-3)


def test_search_end_to_end_finds_planted_atoms_and_feeds_the_subset_regression():
    planted = np.array([3, 17, 29, 41, 50, 58, 63, 70])
    wl, lr, d, coef, target = _problem(72, 5, 4, 24, 32, planted=planted)
    dlr, dco, ddi, dta = dev(lr), dev(coef), dev(d), dev(target)
    rng = np.random.default_rng(8)
    samples = np.sort(rng.choice(wl.npix, size=4000, replace=False)).astype(np.int64)    # the paper samples its LASSO features
    G, b, hh = sr.sr_selection_gram(dlr, dco, ddi, dta, dev(samples), 4, 5)
    nrows = samples.size * wl.c
    idx, gamma, trace = sr.sr_selection_search(G, b, hh, nrows, 8 / 72, 16 / 72, 0.0, 1e-9)
    oG, ob, ohh = oracle.selection_gram(lr, coef, d, target, samples, 4, 5)
    want_idx, want_gamma, want_trace = oracle.selection_search(oG, ob, ohh, nrows, 8 / 72, 16 / 72, 0.0, 1e-9, tol=1e-9, max_sweeps=2000)
    np.testing.assert_array_equal(host(idx), planted)
    np.testing.assert_array_equal(want_idx, planted)
    assert np.abs(host(gamma) - want_gamma).max() <= 1e-3 * np.abs(want_gamma).max()
    np.testing.assert_array_equal(host(trace)[:, 2], want_trace[:, 2])
    # the search's output is the input of the paper's inference-time rule
    out = sr.sr_dict_regress_selected(dlr, dco, idx.contiguous(), gamma.contiguous(), ddi, 4, 5, 8, sr.SR_IDX_GLOBAL)
    want = oracle.dict_regress_selected(lr, coef, host(idx), host(gamma), d, 4, 5, 8, flags=oracle.IDX_GLOBAL)
    assert np.abs(host(out) - want).max() <= TOL_F16
    assert np.mean((host(out) - target) ** 2) <= 0.03 * np.mean(target.astype(np.float64) ** 2)   # eight atoms of 72 keep the image
    assert sr.sr_device_status() == 0
