"""Pins the fp64 CPU oracle to things other than itself.

Each test ties one part of `oracle/` to a fact fixed by the paper's definitions
(Eq. 2-3: y_i = (Phi_i D) B_i^T; Section III-B: taps with the same index are
multiplied, then summed) or by mathematics: exact rational fixtures, a library
resize, a library cross-correlation, algebraic identities and brute force.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as TF

import oracle
import sr_inputs

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
rng = np.random.default_rng(12345)


def _read_rows(name):
    rows = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            parts = line.split()
            rows.setdefault(parts[0], []).append(parts[1:])
    return rows


def _torch_bicubic(lr, r):
    return TF.interpolate(torch.from_numpy(lr).double(), scale_factor=r, mode="bicubic", align_corners=False).numpy()


def _library_dense(lr, coef, dict_, r, k):
    """Phi (D B^T): library resize, replicate pad, library cross-correlation per atom, then combine."""
    U = torch.from_numpy(_torch_bicubic(lr, r))
    n, c, H, W = U.shape
    D = dict_.shape[0]
    p = (k - 1) // 2
    Upad = TF.pad(U.reshape(n * c, 1, H, W), (p, p, p, p), mode="replicate")
    resp = TF.conv2d(Upad, torch.from_numpy(dict_).double().reshape(D, 1, k, k))  # [n*c, D, H, W]
    resp = resp.reshape(n, c, D, H, W)
    phi = torch.from_numpy(coef.astype(np.float64))  # [n, D, H, W]
    return (resp * phi[:, None]).sum(dim=2).numpy()


# ---------------------------------------------------------------- bicubic (stage 1)

@pytest.mark.parametrize("r", [2, 3, 4])
def test_bicubic_closed_form_weights(r):
    """An impulse at LR column q spreads into HR columns with the closed-form phase weights."""
    rows = [row for row in _read_rows("bicubic_weights.txt")[str(r)]]
    h, w = 9, 9
    q = 4
    lr = np.zeros((1, 1, h, w), np.float32)
    lr[0, 0, :, q] = 1.0  # constant along y, impulse along x: U[Y][X] = weight of column q at X
    U = oracle.bicubic_upsample(lr, r)[0, 0]
    for row in rows:
        ph, base = int(row[0]), int(row[1])
        wts = [Fraction(v) for v in row[2:]]
        for qq in range(2, 7):
            X = qq * r + ph
            first = qq + base
            tap = q - first
            expect = float(wts[tap]) if 0 <= tap < 4 else 0.0
            assert abs(U[h * r // 2, X] - expect) < 1e-14, (r, ph, qq)  # (X+1/2)/3 is inexact in fp64
    # and transposed: impulse along y
    lr = np.zeros((1, 1, h, w), np.float32)
    lr[0, 0, q, :] = 1.0
    Ut = oracle.bicubic_upsample(lr, r)[0, 0]
    np.testing.assert_allclose(Ut, U.T, atol=1e-15)


@pytest.mark.parametrize("r,h,w", [(2, 5, 7), (3, 6, 4), (4, 3, 9), (2, 1, 1), (4, 2, 1)])
def test_bicubic_matches_library_resize(r, h, w):
    lr = rng.random((2, 3, h, w), dtype=np.float32)
    np.testing.assert_allclose(oracle.bicubic_upsample(lr, r), _torch_bicubic(lr, r), atol=2e-15)


def test_scale3_centre_pixels_copy_lr():
    lr = rng.random((1, 2, 6, 5), dtype=np.float32)
    U = oracle.bicubic_upsample(lr, 3)
    np.testing.assert_array_equal(U[:, :, 1::3, 1::3], lr.astype(np.float64))


# ---------------------------------------------------------------- worked example (stages 1-4)

def _worked_inputs():
    lr = np.array([[[[0.0, 0.25], [0.5, 1.0]]]], np.float32)
    dict_ = np.zeros((2, 9), np.float32)
    dict_[0, 4] = 1.0
    coef = np.zeros((1, 2, 4, 4), np.float32)
    coef[0, 0] = 0.5
    coef[0, 1] = (4 * np.arange(4)[:, None] + np.arange(4)[None, :]) / 16.0
    return lr, dict_, coef


def test_worked_example_exact_rationals():
    rows = _read_rows("worked_example_4x4.txt")
    U_gold = np.array([[float(Fraction(v)) for v in rows[f"U{i}"][0]] for i in range(4)])
    lr, dict_, coef = _worked_inputs()
    np.testing.assert_allclose(oracle.bicubic_upsample(lr, 2)[0, 0], U_gold, atol=1e-15)
    # dict[1] = 1/9 is not exact in fp32: build the expectation from the fp32 value actually passed in.
    ninth = np.float32(1.0 / 9.0)
    dict_[1, :] = ninth
    y_gold = np.empty((4, 4))
    for Y in range(4):
        for X in range(4):
            y = Fraction(rows[f"y{Y}"][0][X])
            u = Fraction(rows[f"U{Y}"][0][X])
            box9 = (y - u / 2) / Fraction(4 * Y + X, 16) * 9 if (4 * Y + X) else Fraction(0)
            y_gold[Y, X] = float(u / 2 + Fraction(4 * Y + X, 16) * box9 * Fraction(float(ninth)))
    y = oracle.dict_regress_dense(lr, coef, dict_, 2, 3)[0, 0]
    np.testing.assert_allclose(y, y_gold, atol=1e-15)
    # printed decimals of the example (10 digits)
    assert abs(y[0, 0] - (-0.0381603241)) < 1e-8 and abs(y[1, 1] - 0.1682085726) < 1e-8
    assert abs(y[3, 3] - 1.4987112681) < 1e-8
    yc = oracle.dict_regress_dense(lr, coef, dict_, 2, 3, flags=oracle.CLAMP01)[0, 0]
    assert yc[0, 0] == 0.0 and yc[3, 2] == 1.0 and yc[3, 3] == 1.0
    np.testing.assert_array_equal(yc, np.clip(y, 0.0, 1.0))


def test_selection_worked_example():
    phi = np.array([0.5, -0.5, 0.25, 0.5, -0.125, 0.25], np.float32).reshape(1, 6, 1, 1)
    for dt in (np.float32, np.float16):
        assert oracle.dict_select(phi.astype(dt), 3).ravel().tolist() == [0, 1, 3]
        assert oracle.dict_select(phi.astype(dt), 4).ravel().tolist() == [0, 1, 3, 2]
        assert oracle.dict_select(phi.astype(dt), 5).ravel().tolist() == [0, 1, 3, 2, 5]


# ---------------------------------------------------------------- library formulation Phi (D B^T)

@pytest.mark.parametrize("r,k,D,dt", [(2, 5, 6, np.float32), (3, 3, 2, np.float16), (4, 7, 5, np.float16), (2, 1, 3, np.float32)])
def test_dense_matches_library_cross_correlation(r, k, D, dt):
    wl = sr_inputs.Workload("t", 2, 3, 5, 6, r, D=D, k=k, coef_dtype="f16" if dt == np.float16 else "f32")
    lr, dict_, coef = sr_inputs.make_inputs(wl, seed=7)
    # asymmetric atoms so that a flipped or transposed tap order cannot pass
    dict_ = (dict_ + rng.normal(0, 0.1, dict_.shape)).astype(np.float32)
    got = oracle.dict_regress_dense(lr, coef, dict_, r, k)
    np.testing.assert_allclose(got, _library_dense(lr, coef, dict_, r, k), atol=1e-13)


# ---------------------------------------------------------------- identities

def test_delta_atom_one_hot_reproduces_bicubic():
    wl = sr_inputs.Workload("t", 1, 3, 6, 5, 3, D=6, k=5, coef_dtype="f16")
    lr, dict_, _ = sr_inputs.make_inputs(wl)
    dict_[0] = 0
    dict_[0, 12] = 1.0
    coef = np.zeros((1, 6, wl.H, wl.W), np.float16)
    coef[:, 0] = 1.0
    U = _torch_bicubic(lr, 3)
    np.testing.assert_allclose(oracle.dict_regress_dense(lr, coef, dict_, 3, 5), U, atol=2e-15)
    for s in (1, 2, 6):
        np.testing.assert_allclose(oracle.dict_regress_selected(lr, coef, None, None, dict_, 3, 5, s), U, atol=2e-15)
    sub = np.array([0, 3], np.uint8)
    got = oracle.dict_regress_selected(lr, coef, sub, None, dict_, 3, 5, 2, flags=oracle.IDX_GLOBAL)
    np.testing.assert_allclose(got, U, atol=2e-15)


def test_constant_image_stays_constant():
    wl = sr_inputs.Workload("t", 1, 3, 4, 7, 2, D=8, k=5, coef_dtype="f32")
    _, dict_, coef = sr_inputs.make_inputs(wl)
    lr = np.full((1, 3, 4, 7), 0.375, np.float32)
    coef = coef.astype(np.float64)
    coef /= coef.sum(axis=1, keepdims=True)  # sum_l Phi_l = 1 (up to fp32 storage)
    coef = coef.astype(np.float32)
    out = oracle.dict_regress_dense(lr, coef, dict_, 2, 5)
    expect = 0.375 * np.einsum("ndhw,d->nhw", coef.astype(np.float64), dict_.astype(np.float64).sum(axis=1))
    np.testing.assert_allclose(out, np.broadcast_to(expect[:, None], out.shape), atol=1e-14)
    assert np.abs(out - 0.375).max() < 1e-6  # atoms sum to 1 up to fp32 storage


def test_linearity_in_coefficients_image_and_dictionary():
    wl = sr_inputs.Workload("t", 1, 2, 5, 5, 2, D=4, k=3, coef_dtype="f32")
    lr, dict_, c1 = sr_inputs.make_inputs(wl, seed=1)
    _, _, c2 = sr_inputs.make_inputs(wl, seed=2)
    # 0.5 and 0.25 keep fp32 combinations exact
    f = lambda c_, l_=lr, d_=dict_: oracle.dict_regress_dense(l_, c_, d_, 2, 3)
    np.testing.assert_allclose(f((0.5 * c1 + 0.25 * c2).astype(np.float32)), 0.5 * f(c1) + 0.25 * f(c2), atol=1e-7)
    exact1 = (np.round(c1 * 1024) / 1024).astype(np.float32)
    exact2 = (np.round(c2 * 1024) / 1024).astype(np.float32)
    np.testing.assert_allclose(f(0.5 * exact1 + 0.25 * exact2), 0.5 * f(exact1) + 0.25 * f(exact2), atol=1e-14)
    lr2 = (np.round(sr_inputs.make_lr(wl, seed=3) * 256) / 256).astype(np.float32)
    lr1 = (np.round(lr * 256) / 256).astype(np.float32)
    np.testing.assert_allclose(f(exact1, 0.5 * lr1 + 0.25 * lr2), 0.5 * f(exact1, lr1) + 0.25 * f(exact1, lr2), atol=1e-14)
    d1 = (np.round(dict_ * 4096) / 4096).astype(np.float32)
    d2 = d1[::-1].copy()
    np.testing.assert_allclose(f(exact1, lr1, 0.5 * d1 + 0.25 * d2), 0.5 * f(exact1, lr1, d1) + 0.25 * f(exact1, lr1, d2), atol=1e-14)


def test_atom_permutation_leaves_dense_unchanged():
    wl = sr_inputs.Workload("t", 1, 1, 4, 4, 2, D=6, k=3, coef_dtype="f16")
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    perm = np.array([3, 0, 5, 1, 4, 2])
    a = oracle.dict_regress_dense(lr, coef, dict_, 2, 3)
    b = oracle.dict_regress_dense(lr, coef[:, perm].copy(), dict_[perm].copy(), 2, 3)
    np.testing.assert_allclose(a, b, atol=1e-14)


def test_shift_equivariance_in_the_interior():
    r, k = 2, 3
    lr = rng.random((1, 1, 10, 12), dtype=np.float32)
    wl = sr_inputs.Workload("t", 1, 1, 10, 12, r, D=3, k=k, coef_dtype="f32")
    _, dict_, coef = sr_inputs.make_inputs(wl)
    a = oracle.dict_regress_dense(lr, coef, dict_, r, k)
    b = oracle.dict_regress_dense(np.roll(lr, 1, axis=3), np.roll(coef, r, axis=3), dict_, r, k)
    m = 4 * r  # stay away from the borders the roll wraps around / the clamp touches
    np.testing.assert_allclose(np.roll(a, r, axis=3)[..., m:-m, m:-m], b[..., m:-m, m:-m], atol=1e-14)


# ---------------------------------------------------------------- selection

def _brute_topk(coef, s):
    n, D, H, W = coef.shape
    mag = np.abs(coef.astype(np.float64))
    out = np.empty((n, s, H, W), np.uint8)
    for f in range(n):
        for y in range(H):
            for x in range(W):
                order = sorted(range(D), key=lambda l: (-mag[f, l, y, x], l))
                out[f, :, y, x] = order[:s]
    return out


@pytest.mark.parametrize("dt", [np.float16, np.float32])
def test_select_matches_brute_force_with_ties(dt):
    wl = sr_inputs.Workload("t", 2, 1, 3, 4, 2, D=12, k=3, coef_dtype="f16" if dt == np.float16 else "f32")
    coef = sr_inputs.make_coef(wl)
    coef = (np.round(coef.astype(np.float32) * 16) / 16).astype(dt)  # coarse grid: many exact ties, +/- pairs, zeros
    coef[0, 3, 0, 0] = -0.0
    assert (np.abs(coef[:, :-1]) == np.abs(coef[:, 1:])).any()
    for s in (1, 5, 12):
        np.testing.assert_array_equal(oracle.dict_select(coef, s), _brute_topk(coef, s))


def test_select_prefix_and_permutation_and_values():
    wl = sr_inputs.Workload("t", 1, 1, 4, 4, 2, D=16, k=3, coef_dtype="f16")
    coef = sr_inputs.make_coef(wl)
    full, sel = oracle.dict_select(coef, 16, want_sel=True)
    assert (np.sort(full, axis=1) == np.arange(16, dtype=np.uint8)[None, :, None, None]).all()
    for s in (1, 4, 8):
        np.testing.assert_array_equal(oracle.dict_select(coef, s), full[:, :s])
    np.testing.assert_array_equal(sel, np.take_along_axis(coef.astype(np.float64), full.astype(np.int64), axis=1))
    assert (np.abs(sel[:, :-1]) >= np.abs(sel[:, 1:])).all()


def test_selected_equals_dense_when_s_is_D():
    wl = sr_inputs.Workload("t", 2, 3, 4, 5, 2, D=6, k=5, coef_dtype="f16")
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    dense = oracle.dict_regress_dense(lr, coef, dict_, 2, 5)
    idx, sel = oracle.dict_select(coef, 6, want_sel=True)
    np.testing.assert_allclose(oracle.dict_regress_selected(lr, coef, None, None, dict_, 2, 5, 6), dense, atol=1e-14)
    np.testing.assert_allclose(oracle.dict_regress_selected(lr, coef, idx, None, dict_, 2, 5, 6), dense, atol=1e-14)
    comp = oracle.dict_regress_selected(lr, sel.astype(np.float16), idx, None, dict_, 2, 5, 6, flags=oracle.COEF_COMPACT)
    np.testing.assert_allclose(comp, dense, atol=1e-14)


def test_selected_equals_dense_on_masked_coefficients():
    """Keeping s atoms per pixel = dense regression with every other coefficient set to zero."""
    wl = sr_inputs.Workload("t", 1, 3, 5, 4, 3, D=10, k=3, coef_dtype="f32")
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    s = 4
    idx = _brute_topk(coef, s)
    masked = np.zeros_like(coef)
    np.put_along_axis(masked, idx.astype(np.int64), np.take_along_axis(coef, idx.astype(np.int64), axis=1), axis=1)
    want = _library_dense(lr, masked, dict_, 3, 3)
    np.testing.assert_allclose(oracle.dict_regress_selected(lr, coef, None, None, dict_, 3, 3, s), want, atol=1e-13)
    np.testing.assert_allclose(oracle.dict_regress_selected(lr, coef, idx, None, dict_, 3, 3, s), want, atol=1e-13)
    sel = np.take_along_axis(coef, idx.astype(np.int64), axis=1)
    got = oracle.dict_regress_selected(lr, sel, idx, None, dict_, 3, 3, s, flags=oracle.COEF_COMPACT)
    np.testing.assert_allclose(got, want, atol=1e-13)


def test_global_subset_equals_dense_on_sub_dictionary():
    wl = sr_inputs.Workload("t", 2, 3, 4, 4, 2, D=9, k=5, coef_dtype="f16")
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    S = np.array([7, 2, 5], np.uint8)
    gamma = np.array([0.5, 2.0, -1.25], np.float32)
    sub_coef = (coef[:, S.astype(int)].astype(np.float64) * gamma[None, :, None, None])
    want = _library_dense(lr, sub_coef, dict_[S.astype(int)], 2, 5)
    got = oracle.dict_regress_selected(lr, coef, S, gamma, dict_, 2, 5, 3, flags=oracle.IDX_GLOBAL)
    np.testing.assert_allclose(got, want, atol=1e-13)
    compact = coef[:, S.astype(int)].copy()
    got = oracle.dict_regress_selected(lr, compact, S, gamma, dict_, 2, 5, 3, flags=oracle.IDX_GLOBAL | oracle.COEF_COMPACT)
    np.testing.assert_allclose(got, want, atol=1e-13)
    got = oracle.dict_regress_selected(lr, coef, S, None, dict_, 2, 5, 3, flags=oracle.IDX_GLOBAL)
    np.testing.assert_allclose(got, _library_dense(lr, coef[:, S.astype(int)].astype(np.float64), dict_[S.astype(int)], 2, 5), atol=1e-13)


# ---------------------------------------------------------------- sampled evaluation and edge cases

def test_sampled_evaluation_matches_full_frame():
    wl = sr_inputs.Workload("t", 2, 3, 6, 7, 2, D=8, k=5, coef_dtype="f16")
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    samples = rng.choice(wl.npix, size=40, replace=False).astype(np.int64)
    samples[:4] = [0, wl.W - 1, wl.H * wl.W - 1, wl.npix - 1]
    f, pix = samples // (wl.H * wl.W), samples % (wl.H * wl.W)
    dense = oracle.dict_regress_dense(lr, coef, dict_, 2, 5, flags=oracle.CLAMP01)
    got = oracle.regress_at("dense", lr, coef, None, None, dict_, samples, 2, 5, flags=oracle.CLAMP01)
    np.testing.assert_allclose(got, dense.reshape(2, 3, -1)[f, :, pix], atol=1e-14)
    sel = oracle.dict_regress_selected(lr, coef, None, None, dict_, 2, 5, 3)
    got = oracle.regress_at("selected", lr, coef, None, None, dict_, samples, 2, 5, s=3)
    np.testing.assert_allclose(got, sel.reshape(2, 3, -1)[f, :, pix], atol=1e-14)
    idx = oracle.dict_select(coef, 3)
    np.testing.assert_array_equal(oracle.dict_select_at(coef, samples, 3), idx.reshape(2, 3, -1)[f, :, pix])


def test_one_pixel_frame_and_k1():
    lr = np.array([[[[0.625]]]], np.float32)
    dict_ = np.array([[2.0], [-1.0]], np.float32)
    coef = np.array([0.5, 0.25], np.float32).reshape(1, 2, 1, 1)
    assert oracle.dict_regress_dense(lr, coef, dict_, 1, 1)[0, 0, 0, 0] == 0.625 * (0.5 * 2.0 - 0.25)
    out = oracle.dict_regress_dense(np.full((1, 1, 1, 1), 0.5, np.float32), np.ones((1, 1, 2, 2), np.float32),
                                    np.full((1, 9), 1 / 8, np.float32), 2, 3)
    np.testing.assert_allclose(out, 0.5 * 9 / 8, atol=1e-15)


def test_argument_errors():
    lr = np.zeros((1, 1, 2, 2), np.float32)
    with pytest.raises(ValueError):
        oracle.dict_regress_dense(lr, np.zeros((1, 2, 4, 4), np.float32), np.zeros((2, 4), np.float32), 2, 2)  # even k
    with pytest.raises(ValueError):
        oracle.dict_select(np.zeros((1, 2, 4, 4), np.float32), 3)  # s > D


# ---------------------------------------------------------------- generator sanity (inputs only, no method arithmetic)

def test_generator_f16_rounding_matches_numpy():
    x = np.concatenate([rng.normal(0, 0.05, 20000), rng.normal(0, 1e-6, 2000), rng.normal(0, 3e4, 2000),
                        [0.0, -0.0, 65504, 65519.9, 65520, 1e9, 2.0 ** -25, 2.0 ** -25 * 1.0001, 2.0 ** -24, 6.1e-5]])
    x = x.astype(np.float32)
    with np.errstate(over="ignore"):
        want = x.astype(np.float16)
    got = sr_inputs.round_f16(x)
    np.testing.assert_array_equal(got.view(np.uint16), want.view(np.uint16))


def test_generator_distributions_and_dictionary():
    wl = sr_inputs.Workload("t", 1, 3, 32, 32, 2, D=72, k=5, coef_dtype="f32")
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    assert lr.min() >= 0 and lr.max() < 1 and abs(lr.mean() - 0.5) < 0.02
    assert abs(coef.mean() - 1 / 72) < 1e-3 and abs(coef.std() - 0.05) < 1e-3
    np.testing.assert_allclose(dict_.sum(axis=1), 1.0, atol=1e-6)
    assert dict_.min() >= 0 and dict_.max() <= 1.0
    assert (dict_[36:, 12] == 0).all()           # difference of two peak-1 Gaussians vanishes at the centre
    assert (dict_[:36, 12] == dict_[:36].max(axis=1)).all()
    lr2, _, coef2 = sr_inputs.make_inputs(wl)
    np.testing.assert_array_equal(coef, coef2)
    half = sr_inputs.make_coef(sr_inputs.Workload("t", 1, 3, 32, 32, 2, coef_dtype="f16"))
    np.testing.assert_array_equal(half, sr_inputs.round_f16(coef))


def test_binary16_widening_every_bit_pattern():
    """The oracle widens binary16 coefficients itself (sign, exponent, mantissa; subnormals, infinities, NaN). Every one
    of the 65536 bit patterns is pinned against numpy's own float16 -> float64 conversion, through the two routes a
    coefficient takes: the selected values (`sel` of the selection) and the regression (a 1 x 1 unit atom on a
    constant unit image returns the coefficient itself)."""
    bits = np.arange(65536, dtype=np.uint16)
    coef = bits.view(np.float16).reshape(1, 1, 256, 256)
    want = coef.astype(np.float64)
    _, sel = oracle.dict_select(coef, 1, want_sel=True)
    finite = np.isfinite(want)
    np.testing.assert_array_equal(sel[finite], want[finite])
    np.testing.assert_array_equal(np.isnan(sel), np.isnan(want))
    np.testing.assert_array_equal(sel[np.isinf(want)], want[np.isinf(want)])
    assert np.array_equal(np.signbit(sel[finite]), np.signbit(want[finite]))      # -0 keeps its sign
    # subnormals and the largest finite value, by hand
    for b, v in ((0x0001, 2.0 ** -24), (0x03FF, 1023 * 2.0 ** -24), (0x0400, 2.0 ** -14), (0x7BFF, 65504.0), (0xFBFF, -65504.0)):
        assert sel.reshape(-1)[b] == v
    lr = np.ones((1, 1, 256, 256), np.float32)
    out = oracle.dict_regress_dense(lr, coef, np.ones((1, 1), np.float32), 1, 1)
    np.testing.assert_array_equal(out[0][finite[0]], want[0][finite[0]])


def test_eight_bit_output_codes():
    """SR_OUT_U8 in the oracle: the code of the clamped value on the 255-step grid. Pinned by the worked 4 x 4 example
    (its printed values times 255, rounded by hand: -0.0382 -> 0, 0.1682 -> 43, 0.5123 -> 131, 1.4987 -> 255), by
    numpy's rint on the oracle's own unquantised output, and by the round-half-even rule on exact ties."""
    lr = np.array([[[[0.0, 0.25], [0.5, 1.0]]]], np.float32)
    d = np.zeros((2, 9), np.float32)
    d[0, 4] = 1.0
    d[1, :] = 1.0 / 9.0
    coef = np.zeros((1, 2, 4, 4), np.float32)
    coef[0, 0] = 0.5
    coef[0, 1] = (4 * np.arange(4)[:, None] + np.arange(4)[None, :]) / 16.0
    codes = oracle.dict_regress_dense(lr, coef, d, 2, 3, flags=oracle.OUT_U8)[0, 0]
    assert codes[0, 0] == 0 and codes[1, 1] == 43 and codes[2, 1] == 131 and codes[3, 3] == 255
    plain = oracle.dict_regress_dense(lr, coef, d, 2, 3)
    np.testing.assert_array_equal(codes, np.rint(255.0 * np.clip(plain[0, 0], 0.0, 1.0)))
    # exact ties: 0.5 / 255 and 1.5 / 255 are not representable, so build ties through the atom weight instead:
    # a 1 x 1 unit atom on a constant image of value 1 returns the coefficient; x.5 / 255 * 255 is a tie only in exact
    # arithmetic, so check the integers around it and the monotone staircase
    lr1 = np.ones((1, 1, 1, 256), np.float32)
    co = (np.arange(256, dtype=np.float64) / 255.0).astype(np.float32).reshape(1, 1, 1, 256)
    q = oracle.dict_regress_dense(lr1, co, np.ones((1, 1), np.float32), 1, 1, flags=oracle.OUT_U8)[0, 0, 0]
    np.testing.assert_array_equal(q, np.arange(256))
    wl = sr_inputs.Workload("t", 1, 3, 6, 7, 2, D=6, k=3, coef_dtype="f16")
    lr, dd, cf = sr_inputs.make_inputs(wl)
    q = oracle.dict_regress_selected(lr, cf, None, None, dd, 2, 3, 2, flags=oracle.OUT_U8)
    v = oracle.dict_regress_selected(lr, cf, None, None, dd, 2, 3, 2)
    np.testing.assert_array_equal(q, np.rint(255.0 * np.clip(v, 0.0, 1.0)))
    assert q.min() >= 0 and q.max() <= 255


def test_luma_only_regression():
    """LUMA_ONLY in the oracle (filter the BT.601 luma of the up-sampled image, keep the up-sampled chroma), pinned by:
    the composition out = U + (regression of the luma image - luma of U) built from the pinned one-channel regression
    and bicubic (stage 1 is linear, so up-sampling the luma of the LR image is the luma of the up-sampled image);
    chroma differences that equal those of U; a grey image, where it is the ordinary regression; the delta atom."""
    wy = np.array([0.299, 0.587, 0.114])
    wl = sr_inputs.Workload("t", 2, 3, 7, 9, 3, D=6, k=5, coef_dtype="f16")
    lr, d, coef = sr_inputs.make_inputs(wl)
    d = (d + np.random.default_rng(1).normal(0, 0.1, d.shape)).astype(np.float32)
    out = oracle.dict_regress_dense(lr, coef, d, 3, 5, flags=oracle.LUMA_ONLY)
    U = oracle.bicubic_upsample(lr, 3)
    UY = np.tensordot(wy, U, axes=([0], [1]))[:, None]                       # [n][1][H][W]
    lrY = np.tensordot(wy, lr.astype(np.float64), axes=([0], [1]))[:, None]
    regY = oracle.dict_regress_dense(lrY.astype(np.float32), coef, d, 3, 5)  # the luma image through the one-channel path
    want = U + (regY - UY)
    assert np.abs(out - want).max() <= 5e-7                                  # fp32 rounding of the luma LR image only
    outY = np.tensordot(wy, out, axes=([0], [1]))[:, None]
    assert np.abs((out - outY) - (U - UY)).max() <= 1e-12                    # chroma differences untouched
    # selected modes go through the same pixel routine
    sel = oracle.dict_regress_selected(lr, coef, None, None, d, 3, 5, 2, flags=oracle.LUMA_ONLY)
    regY = oracle.dict_regress_selected(lrY.astype(np.float32), coef, None, None, d, 3, 5, 2)
    assert np.abs(sel - (U + (regY - UY))).max() <= 5e-7
    # grey image: luma = every channel, so nothing changes
    grey = np.repeat(lr[:, :1], 3, axis=1)
    a = oracle.dict_regress_dense(grey, coef, d, 3, 5, flags=oracle.LUMA_ONLY)
    b = oracle.dict_regress_dense(grey, coef, d, 3, 5)
    assert np.abs(a - b).max() <= 1e-12
    # delta atom, one-hot coefficients: the up-sampled image itself
    dd = np.zeros_like(d)
    dd[0, 12] = 1.0
    one = np.zeros_like(coef)
    one[:, 0] = 1.0
    assert np.abs(oracle.dict_regress_dense(lr, one, dd, 3, 5, flags=oracle.LUMA_ONLY) - U).max() <= 1e-12
    with pytest.raises(ValueError):
        oracle.dict_regress_dense(lr[:, :2], coef, d, 3, 5, flags=oracle.LUMA_ONLY)
