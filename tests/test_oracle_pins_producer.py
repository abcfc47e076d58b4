"""Pins of the oracle's producer of Phi (last convolution + pixel-shuffle; Section II-A, stage 2 tail) and of the
regression that takes Phi from it.

The coefficient tensor is pinned against a library convolution and a library sub-pixel shuffle (fp64, zero padding),
and by hand-built cases: a 1x1 convolution with one-hot weights is a pure channel shuffle whose output is known in
closed form; a single tap at an off-centre position shifts the feature map (sign of the shift, padding, row/column
order); the bias alone gives constant planes. The regression is pinned by composition with the already pinned dense
regression and global-subset regression fed with that tensor.
"""
import numpy as np
import pytest
import torch

import oracle
import sr_inputs


def _inputs(n=2, h=6, w=7, r=2, D=5, k=3, cin=4, kc=3, seed=3):
    wl = sr_inputs.Workload("t", n, 3, h, w, r, D=D, k=k)
    lr, dict_, _ = sr_inputs.make_inputs(wl, seed=seed)
    feat, wconv, bias = sr_inputs.make_producer(wl, cin=cin, kc=kc, seed=seed)
    dict_ = (dict_ + np.random.default_rng(seed).normal(0, 0.1, dict_.shape)).astype(np.float32)
    return wl, lr, dict_, feat, wconv, bias


@pytest.mark.parametrize("r,kc,cin", [(2, 3, 4), (3, 3, 2), (4, 1, 8), (1, 3, 3), (2, 5, 2)])
def test_coefficients_match_library_convolution_and_shuffle(r, kc, cin):
    wl, lr, dict_, feat, wconv, bias = _inputs(r=r, kc=kc, cin=cin)
    phi = oracle.producer_coef(feat, wconv, bias, r)
    x = torch.from_numpy(feat.astype(np.float64)).permute(0, 3, 1, 2)            # channels first for the library
    y = torch.nn.functional.conv2d(x, torch.from_numpy(wconv.astype(np.float64)), torch.from_numpy(bias.astype(np.float64)),
                                   padding=kc // 2)
    want = torch.nn.functional.pixel_shuffle(y, r).numpy()
    assert phi.shape == want.shape == (wl.n, wl.D, wl.H, wl.W)
    assert np.abs(phi - want).max() <= 1e-12
    no_bias = oracle.producer_coef(feat, wconv, None, r)
    assert np.abs(no_bias + _bias_planes(bias, wl) - phi).max() <= 1e-12

def _bias_planes(bias, wl):
    """bias[l r^2 + ry r + rx] laid out as the planes the shuffle makes of it: [1][D][H][W]."""
    r = wl.scale
    b = bias.astype(np.float64).reshape(wl.D, r, r)
    return np.tile(b, (1, wl.h, wl.w))[None]


def test_one_hot_1x1_convolution_is_a_channel_shuffle():
    r, D = 2, 3
    wl = sr_inputs.Workload("t", 1, 3, 4, 5, r, D=D, k=3)
    cin = D * r * r
    feat = sr_inputs.round_f16(np.random.default_rng(0).normal(size=(1, wl.h, wl.w, cin)).astype(np.float32))
    wconv = np.eye(cin, dtype=np.float32).reshape(cin, cin, 1, 1)
    phi = oracle.producer_coef(feat, wconv, None, r)
    for l in range(D):
        for Y in range(wl.H):
            for X in range(wl.W):
                assert phi[0, l, Y, X] == float(feat[0, Y // r, X // r, l * r * r + (Y % r) * r + (X % r)])


def test_single_off_centre_tap_shifts_with_zero_padding():
    """weight 1 at tap (dy, dx) = (0, 2) of a 3x3 kernel reads feat[y - 1][x + 1]; outside the map it reads zero."""
    wl = sr_inputs.Workload("t", 1, 3, 5, 6, 1, D=1, k=3)
    feat = sr_inputs.round_f16(np.random.default_rng(1).uniform(1, 2, size=(1, wl.h, wl.w, 2)).astype(np.float32))
    wconv = np.zeros((1, 2, 3, 3), dtype=np.float32)
    wconv[0, 1, 0, 2] = 1.0
    phi = oracle.producer_coef(feat, wconv, None, 1)[0, 0]
    f = feat[0, :, :, 1].astype(np.float64)
    want = np.zeros_like(f)
    want[1:, :-1] = f[:-1, 1:]
    assert np.array_equal(phi, want)


def test_bias_alone_gives_phase_constant_planes():
    wl, lr, dict_, feat, wconv, bias = _inputs(r=3, D=4)
    phi = oracle.producer_coef(feat, np.zeros_like(wconv), bias, 3)
    assert np.array_equal(phi, np.broadcast_to(_bias_planes(bias, wl), phi.shape))


@pytest.mark.parametrize("r,k,kc", [(2, 3, 3), (3, 5, 1), (4, 3, 3)])
def test_regression_is_the_pinned_dense_regression_on_the_produced_tensor(r, k, kc):
    wl, lr, dict_, feat, wconv, bias = _inputs(r=r, k=k, kc=kc, D=6)
    phi = oracle.producer_coef(feat, wconv, bias, r)
    for fl in (0, oracle.CLAMP01, oracle.UPSAMPLE_BILINEAR, oracle.LUMA_ONLY, oracle.OUT_U8):
        got = oracle.producer_regress(lr, feat, wconv, bias, dict_, r, k, flags=fl)
        want = oracle.dict_regress_dense(lr, phi.astype(np.float32), dict_, r, k, flags=fl)
        if fl == oracle.OUT_U8:
            assert np.abs(got - want).max() <= 1 and np.mean(got != want) < 1e-3        # a code may flip at a boundary
        else:
            assert np.abs(got - want).max() <= 2e-7                                     # fp32 rounding of the stored tensor
    # something was actually regressed: the result differs from plain up-sampling
    assert np.abs(oracle.producer_regress(lr, feat, wconv, bias, dict_, r, k) - oracle.bicubic_upsample(lr, r)).max() > 1e-2


def test_global_subset_is_the_pinned_subset_regression():
    wl, lr, dict_, feat, wconv, bias = _inputs(r=2, k=3, D=7)
    phi = oracle.producer_coef(feat, wconv, bias, 2).astype(np.float32)
    S = np.array([5, 0, 3], dtype=np.uint8)
    gamma = np.array([1.25, -0.5, 0.75], dtype=np.float32)
    got = oracle.producer_regress(lr, feat, wconv, bias, dict_, 2, 3, idx=S, gamma=gamma)
    want = oracle.dict_regress_selected(lr, phi, S, gamma, dict_, 2, 3, 3, flags=oracle.IDX_GLOBAL)
    assert np.abs(got - want).max() <= 2e-7
    ones = oracle.producer_regress(lr, feat, wconv, bias, dict_, 2, 3, idx=S)
    want = oracle.dict_regress_selected(lr, phi, S, None, dict_, 2, 3, 3, flags=oracle.IDX_GLOBAL)
    assert np.abs(ones - want).max() <= 2e-7
    every = oracle.producer_regress(lr, feat, wconv, bias, dict_, 2, 3, idx=np.arange(7, dtype=np.uint8))
    assert np.abs(every - oracle.producer_regress(lr, feat, wconv, bias, dict_, 2, 3)).max() <= 1e-12


def test_generated_coefficients_have_the_benchmark_distribution():
    wl = sr_inputs.Workload("t", 1, 3, 24, 32, 2, D=16, k=3)
    feat, wconv, bias = sr_inputs.make_producer(wl, cin=32, kc=3)
    phi = oracle.producer_coef(feat, wconv, bias, 2)[:, :, 4:-4, 4:-4]                 # away from the zero padding
    assert abs(phi.mean() - 1 / 16) < 5e-3 and abs(phi.std() - 0.05) < 6e-3
