"""Pins for the oracle's bilinear up-sampling (stage 1a as the paper words it, Section II-A) and for the regression
calls with that variant selected: a library resize, closed-form phase weights, exact reproduction of affine images
away from the border, the border rule, and the delta-atom identity through stages 1-4.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as TF

import oracle
import sr_inputs

rng = np.random.default_rng(8999)


def _torch_bilinear(lr, r):
    return TF.interpolate(torch.from_numpy(lr).double(), scale_factor=r, mode="bilinear", align_corners=False).numpy()


@pytest.mark.parametrize("r,h,w", [(2, 5, 7), (3, 6, 4), (4, 3, 9), (2, 1, 1), (4, 2, 1), (1, 3, 3)])
def test_bilinear_matches_library_resize(r, h, w):
    lr = rng.random((2, 3, h, w), dtype=np.float32)
    np.testing.assert_allclose(oracle.bilinear_upsample(lr, r), _torch_bilinear(lr, r), atol=2e-15)


@pytest.mark.parametrize("r", [2, 3, 4])
def test_bilinear_closed_form_weights(r):
    """An impulse at LR column q reaches HR column X = q'r + p with weight 1 - t or t, t = frac((2p + 1 - r) / (2r))."""
    h, w, q = 5, 9, 4
    lr = np.zeros((1, 1, h, w), np.float32)
    lr[0, 0, :, q] = 1.0
    U = oracle.bilinear_upsample(lr, r)[0, 0]
    for qq in range(2, 7):
        for p in range(r):
            num = Fraction(2 * p + 1 - r, 2 * r)          # sample point relative to LR column qq
            i0 = qq + (num.numerator // num.denominator)  # floor
            t = num - (num.numerator // num.denominator)
            expect = (1 - t) if i0 == q else (t if i0 + 1 == q else Fraction(0))
            assert abs(U[h * r // 2, qq * r + p] - float(expect)) < 1e-15, (r, p, qq)
    # r = 2 in numbers: phases (1/4, 3/4) and (3/4, 1/4)
    if r == 2:
        np.testing.assert_allclose(U[4, 2 * q - 1: 2 * q + 3], [0.25, 0.75, 0.75, 0.25], atol=0)


@pytest.mark.parametrize("r", [2, 3, 4])
def test_bilinear_reproduces_affine_images_inside(r):
    """Linear interpolation is exact for x[y][x] = a + b y + c x wherever both neighbours exist."""
    h, w = 6, 7
    yy, xx = np.meshgrid(np.arange(h), np.arange(w), indexing="ij")
    lr = (0.25 + 0.125 * yy - 0.0625 * xx).astype(np.float32)[None, None]
    U = oracle.bilinear_upsample(lr, r)[0, 0]
    Y, X = np.meshgrid(np.arange(h * r), np.arange(w * r), indexing="ij")
    sy, sx = (Y + 0.5) / r - 0.5, (X + 0.5) / r - 0.5
    inside = (sy >= 0) & (sy <= h - 1) & (sx >= 0) & (sx <= w - 1)
    want = 0.25 + 0.125 * sy - 0.0625 * sx
    np.testing.assert_allclose(U[inside], want[inside], atol=1e-14)
    # outside, the clamped neighbour is used: the first HR column repeats LR column 0 of the affine image
    np.testing.assert_allclose(U[r:2 * r, 0], (0.25 + 0.125 * sy[r:2 * r, 0]), atol=1e-14)


def test_bilinear_constant_and_range():
    lr = np.full((1, 2, 3, 4), 0.625, np.float32)
    np.testing.assert_array_equal(oracle.bilinear_upsample(lr, 4), np.full((1, 2, 12, 16), 0.625))
    lr = rng.random((1, 1, 5, 5), dtype=np.float32)
    U = oracle.bilinear_upsample(lr, 3)
    assert U.min() >= lr.min() and U.max() <= lr.max()      # a convex combination never overshoots (bicubic does)


def test_delta_atom_reproduces_bilinear_through_all_calls():
    wl = sr_inputs.Workload("t", 1, 3, 6, 5, 3, D=6, k=5, coef_dtype="f16")
    lr, dict_, _ = sr_inputs.make_inputs(wl)
    dict_[0] = 0
    dict_[0, 12] = 1.0
    coef = np.zeros((1, 6, wl.H, wl.W), np.float16)
    coef[:, 0] = 1.0
    U = _torch_bilinear(lr, 3)
    B = oracle.UPSAMPLE_BILINEAR
    np.testing.assert_allclose(oracle.dict_regress_dense(lr, coef, dict_, 3, 5, flags=B), U, atol=2e-15)
    for s in (1, 2, 6):
        np.testing.assert_allclose(oracle.dict_regress_selected(lr, coef, None, None, dict_, 3, 5, s, flags=B), U, atol=2e-15)
    sub = np.array([0, 3], np.uint8)
    got = oracle.dict_regress_selected(lr, coef, sub, None, dict_, 3, 5, 2, flags=oracle.IDX_GLOBAL | B)
    np.testing.assert_allclose(got, U, atol=2e-15)
    # the sampled entry point takes the same flag
    samples = np.array([0, 7, wl.H * wl.W - 1], dtype=np.int64)
    at = oracle.regress_at("dense", lr, coef, None, None, dict_, samples, 3, 5, flags=B)
    full = oracle.dict_regress_dense(lr, coef, dict_, 3, 5, flags=B)
    np.testing.assert_allclose(at, full.reshape(3, -1)[:, samples].T.reshape(at.shape), atol=0)


def test_box_atom_equals_library_correlation_of_bilinear_image():
    """A 3x3 box atom with coefficient 1: out = box filter of the replicate-padded bilinear image."""
    lr = rng.random((1, 2, 4, 5), dtype=np.float32)
    dict_ = np.full((1, 9), 1.0 / 9.0, np.float32)
    coef = np.ones((1, 1, 8, 10), np.float32)
    got = oracle.dict_regress_dense(lr, coef, dict_, 2, 3, flags=oracle.UPSAMPLE_BILINEAR)
    U = torch.from_numpy(_torch_bilinear(lr, 2))
    pad = TF.pad(U, (1, 1, 1, 1), mode="replicate")
    kern = torch.from_numpy(dict_.astype(np.float64)).reshape(1, 1, 3, 3)
    want = TF.conv2d(pad.reshape(2, 1, 10, 12), kern).reshape(1, 2, 8, 10).numpy()
    np.testing.assert_allclose(got, want, atol=1e-14)
