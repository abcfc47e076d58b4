"""Parity of the CUDA library (called through its C ABI) against the fp64 CPU oracle.

Small cases are compared element by element; they span several tiles, ragged tails, every atom size
and both coefficient types. Index outputs must be bit-exact; pixel values within 1e-5 (fp32
coefficients) or 2e-3 (binary16 coefficients) max abs error.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, TOL_F32, dev, host, max_abs_err, signed_asymmetric_dictionary, signed_gamma, tol_for

pytestmark = pytest.mark.gpu


def _wl(n, c, h, w, r, D, k, dt):
    return sr_inputs.Workload("t", n, c, h, w, r, D=D, k=k, coef_dtype=dt)


# ------------------------------------------------------------------ stage 1

@pytest.mark.parametrize("n,c,h,w,r", [(1, 3, 64, 64, 2), (2, 3, 37, 53, 3), (1, 1, 5, 300, 4), (1, 2, 1, 1, 2),
                                       (1, 3, 9, 7, 1), (1, 1, 6, 5, 8), (1, 4, 2, 3, 5), (1, 3, 41, 35, 3), (2, 1, 9, 11, 6),
                                       (1, 2, 13, 10, 5), (1, 1, 7, 9, 7)])
def test_bicubic(n, c, h, w, r):
    lr = sr_inputs.make_lr(_wl(n, c, h, w, r, 1, 1, "f32"))
    got = host(sr.sr_bicubic_upsample(dev(lr), r))
    want = oracle.bicubic_upsample(lr, r)
    assert max_abs_err(got, want) <= 1e-6


# ------------------------------------------------------------------ dense

DENSE_CASES = [
    # n, c, h, w, r, D, k, dtype
    (1, 3, 64, 64, 2, 72, 5, "f32"),      # cfg0 in full
    (1, 3, 64, 64, 2, 72, 5, "f16"),
    (2, 3, 33, 50, 4, 72, 5, "f16"),      # ragged in both directions, two frames
    (1, 3, 20, 67, 3, 72, 5, "f16"),
    (1, 1, 40, 24, 2, 16, 3, "f16"),
    (1, 3, 24, 40, 2, 32, 7, "f16"),
    (1, 3, 12, 40, 4, 128, 5, "f16"),
    (1, 3, 10, 24, 2, 256, 3, "f16"),
    (1, 5, 9, 16, 2, 7, 9, "f32"),        # odd atom count, five channels, largest atom
    (1, 3, 7, 5, 3, 3, 1, "f32"),         # 1x1 atoms
    (1, 3, 1, 1, 2, 72, 5, "f16"),        # a single LR pixel
    (1, 3, 3, 100, 4, 72, 5, "f16"),      # HR width 400: not a multiple of 128
    (1, 3, 30, 35, 4, 72, 5, "f16"),      # HR width 140: not a multiple of 8
]


@pytest.mark.parametrize("case", DENSE_CASES, ids=lambda c: "-".join(map(str, c)))
@pytest.mark.parametrize("clamp", [0, 1])
def test_dense(case, clamp):
    n, c, h, w, r, D, k, dt = case
    lr, dict_, coef = sr_inputs.make_inputs(_wl(n, c, h, w, r, D, k, dt))
    if k == 1:  # a difference of Gaussians has no 1x1 form (0/0): use plain seeded weights instead
        dict_ = np.random.default_rng(1).uniform(-1, 1, dict_.shape).astype(np.float32)
    flags = sr.SR_CLAMP01 if clamp else 0
    got = host(sr.sr_dict_regress_dense(dev(lr), dev(coef), dev(dict_), r, k, flags))
    want = oracle.dict_regress_dense(lr, coef, dict_, r, k, flags=flags)
    assert sr.sr_device_status() == 0
    assert max_abs_err(got, want) <= tol_for(coef)


def test_dense_is_deterministic_and_leaves_inputs_alone():
    lr, dict_, coef = sr_inputs.make_inputs(_wl(2, 3, 33, 50, 4, 72, 5, "f16"))
    dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
    a = host(sr.sr_dict_regress_dense(dlr, dco, ddi, 4, 5))
    b = host(sr.sr_dict_regress_dense(dlr, dco, ddi, 4, 5))
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(host(dco), coef)
    np.testing.assert_array_equal(host(dlr), lr)


def test_dense_delta_atom_reproduces_bicubic_on_gpu():
    wl = _wl(1, 3, 20, 48, 4, 72, 5, "f16")
    lr, dict_, _ = sr_inputs.make_inputs(wl)
    dict_[0] = 0
    dict_[0, 12] = 1
    coef = np.zeros((1, 72, wl.H, wl.W), np.float16)
    coef[:, 0] = 1
    got = host(sr.sr_dict_regress_dense(dev(lr), dev(coef), dev(dict_), 4, 5))
    up = host(sr.sr_bicubic_upsample(dev(lr), 4))
    assert max_abs_err(got, up.astype(np.float64)) <= 1e-6
    assert max_abs_err(got, oracle.bicubic_upsample(lr, 4)) <= 1e-6


def test_dense_on_a_side_stream_and_offset_views():
    """Pointers that are element-aligned but not 16-byte aligned still work (general path)."""
    wl = _wl(1, 3, 16, 24, 2, 16, 3, "f16")
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    buf = torch.empty(coef.size + 1, dtype=torch.float16, device="cuda")
    view = buf[1:].view(coef.shape)
    view.copy_(dev(coef))
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        got = sr.sr_dict_regress_dense(dev(lr), view, dev(dict_), 2, 3)
    st.synchronize()
    assert max_abs_err(host(got), oracle.dict_regress_dense(lr, coef, dict_, 2, 3)) <= TOL_F16


# ------------------------------------------------------------------ selection

def _coarse(coef):
    """Quantise to a coarse grid so that exact magnitude ties, +/- pairs and zeros are frequent."""
    return (np.round(coef.astype(np.float32) * 64) / 64).astype(coef.dtype)


@pytest.mark.parametrize("dt", ["f16", "f32"])
@pytest.mark.parametrize("D,s", [(72, 8), (72, 1), (72, 4), (72, 16), (72, 20), (72, 72), (16, 16), (128, 8), (256, 5), (5, 3)])
def test_select_bit_exact(dt, D, s):
    wl = _wl(2, 1, 9, 23, 2, D, 1, dt)
    for coef in (sr_inputs.make_coef(wl), _coarse(sr_inputs.make_coef(wl, seed=5))):
        idx, sel = sr.sr_dict_select(dev(coef), s, want_sel=True)
        want_idx, want_sel = oracle.dict_select(coef, s, want_sel=True)
        np.testing.assert_array_equal(host(idx), want_idx)
        np.testing.assert_array_equal(host(sel).astype(np.float64), want_sel)
        np.testing.assert_array_equal(host(sr.sr_dict_select(dev(coef), s)), want_idx)


def test_select_signed_zero_and_extremes():
    coef = np.zeros((1, 8, 2, 8), np.float16)
    coef[0, 3] = -0.0
    coef[0, 5, 0, :] = [65504, -65504, 6e-8, -6e-8, 1, -1, 0.5, 0]
    coef[0, 6, 0, :] = [-65504, 65504, -6e-8, 6e-8, -1, 1, 0.25, -0.0]
    np.testing.assert_array_equal(host(sr.sr_dict_select(dev(coef), 3)), oracle.dict_select(coef, 3))


# ------------------------------------------------------------------ selected regression

SEL_CASES = [
    (1, 3, 33, 50, 4, 72, 5, "f16", 8),
    (2, 3, 20, 30, 2, 72, 5, "f32", 8),
    (1, 3, 16, 40, 3, 32, 3, "f16", 4),
    (1, 1, 12, 24, 2, 128, 7, "f16", 16),
    (1, 3, 8, 24, 2, 72, 5, "f16", 20),
    (1, 3, 8, 24, 2, 16, 5, "f16", 16),
    # widths that are multiples of 16: the index-listed and compact modes take the tensor-core kernel too
    (1, 3, 24, 64, 2, 72, 5, "f16", 8),
    (1, 3, 20, 36, 4, 32, 3, "f16", 4),
    (2, 3, 9, 40, 2, 128, 5, "f16", 8),
    (1, 3, 10, 24, 2, 20, 5, "f16", 3),
    (1, 2, 40, 72, 4, 72, 3, "f16", 8),
    (1, 3, 7, 168, 2, 6, 7, "f16", 6),
    # 8 < s <= 16: the sixteen-entry list of the in-kernel selection, two rank halves per lane in the listed modes
    (1, 3, 12, 32, 2, 72, 5, "f16", 12),
    (1, 3, 12, 64, 4, 128, 3, "f16", 16),
    (1, 3, 10, 40, 2, 24, 5, "f16", 9),
]


@pytest.mark.parametrize("case", SEL_CASES, ids=lambda c: "-".join(map(str, c)))
def test_selected_all_modes(case):
    n, c, h, w, r, D, k, dt, s = case
    wl = _wl(n, c, h, w, r, D, k, dt)
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    tol = tol_for(coef)
    dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
    want = oracle.dict_regress_selected(lr, coef, None, None, dict_, r, k, s, flags=oracle.CLAMP01)
    # top-s chosen inside the call
    got = host(sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s, sr.SR_CLAMP01))
    assert max_abs_err(got, want) <= tol
    # two-step: select, then regress from the index planes (full tensor, then compact values)
    idx, sel = sr.sr_dict_select(dco, s, want_sel=True)
    got = host(sr.sr_dict_regress_selected(dlr, dco, idx, None, ddi, r, k, s, sr.SR_CLAMP01))
    assert max_abs_err(got, want) <= tol
    got = host(sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, s, sr.SR_CLAMP01 | sr.SR_COEF_COMPACT))
    assert max_abs_err(got, want) <= tol
    # the paper's global subset with re-weights
    rng = np.random.default_rng(3)
    S = rng.choice(D, size=s, replace=False).astype(np.uint8)
    gamma = rng.uniform(0.5, 1.5, size=s).astype(np.float32)
    want = oracle.dict_regress_selected(lr, coef, S, gamma, dict_, r, k, s, flags=oracle.IDX_GLOBAL)
    got = host(sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, s, sr.SR_IDX_GLOBAL))
    assert max_abs_err(got, want) <= tol
    compact = dev(coef[:, S.astype(int)].copy())
    got = host(sr.sr_dict_regress_selected(dlr, compact, dev(S), dev(gamma), ddi, r, k, s,
                                           sr.SR_IDX_GLOBAL | sr.SR_COEF_COMPACT))
    assert max_abs_err(got, want) <= tol
    want = oracle.dict_regress_selected(lr, coef, S, None, dict_, r, k, s, flags=oracle.IDX_GLOBAL)
    got = host(sr.sr_dict_regress_selected(dlr, dco, dev(S), None, ddi, r, k, s, sr.SR_IDX_GLOBAL))
    assert max_abs_err(got, want) <= tol
    assert sr.sr_device_status() == 0


def test_selected_with_s_equal_D_is_dense():
    wl = _wl(1, 3, 16, 24, 2, 16, 5, "f16")
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    a = host(sr.sr_dict_regress_selected(dev(lr), dev(coef), None, None, dev(dict_), 2, 5, 16))
    assert max_abs_err(a, oracle.dict_regress_dense(lr, coef, dict_, 2, 5)) <= TOL_F16


@pytest.mark.parametrize("D,s,w", [(72, 8, 24), (128, 5, 64), (24, 8, 32), (72, 1, 24), (72, 13, 32), (40, 16, 24)])
def test_selected_with_ties(D, s, w):
    wl = _wl(1, 3, 16, w, 2, D, 5, "f16")
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    coef = _coarse(coef)
    want = oracle.dict_regress_selected(lr, coef, None, None, dict_, 2, 5, s)
    got = host(sr.sr_dict_regress_selected(dev(lr), dev(coef), None, None, dev(dict_), 2, 5, s))
    assert max_abs_err(got, want) <= TOL_F16
    # the same pixels through explicit index planes (ties resolved by sr_dict_select) and compact values
    idx, sel = sr.sr_dict_select(dev(coef), s, want_sel=True)
    np.testing.assert_array_equal(host(idx), oracle.dict_select(coef, s))
    got = host(sr.sr_dict_regress_selected(dev(lr), dev(coef), idx, None, dev(dict_), 2, 5, s))
    assert max_abs_err(got, want) <= TOL_F16
    got = host(sr.sr_dict_regress_selected(dev(lr), sel, idx, None, dev(dict_), 2, 5, s, sr.SR_COEF_COMPACT))
    assert max_abs_err(got, want) <= TOL_F16


# ------------------------------------------------------------------ orientation and sign of the taps

SIGNED_CASES = [
    # n, c, h, w, r, D, k, dtype, s
    (1, 3, 24, 64, 2, 72, 5, "f16", 8),    # every mode on the tensor-core kernel
    (2, 3, 33, 50, 4, 72, 5, "f16", 8),    # HR width 200: dense / in-kernel selection / subset on the tensor cores, index planes on the general kernel
    (1, 3, 20, 30, 2, 72, 5, "f32", 8),    # fp32 coefficients: general kernel
    (1, 3, 12, 40, 2, 32, 7, "f16", 4),
    (1, 3, 12, 32, 2, 72, 3, "f16", 12),
    (1, 1, 9, 16, 2, 7, 9, "f32", 3),      # 9 x 9 atoms: general kernel
    (1, 3, 30, 35, 4, 72, 5, "f16", 8),    # HR width 140: general kernel with binary16 coefficients
    (1, 3, 40, 64, 4, 72, 5, "f16", 8),    # several 16-row tiles, two tile columns
]


@pytest.mark.parametrize("case", SIGNED_CASES, ids=lambda c: "-".join(map(str, c)))
def test_signed_asymmetric_dictionary_and_negative_gamma_all_modes(case):
    """Atoms without any symmetry and with both signs, re-weights with both signs: a 180-degree tap flip, a transposed
    patch or a lost sign in the binary16 hi / lo split of the dictionary fails here (it passes with the generator's
    point-symmetric, non-negative atoms)."""
    n, c, h, w, r, D, k, dt, s = case
    wl = _wl(n, c, h, w, r, D, k, dt)
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    dict_ = signed_asymmetric_dictionary(dict_)
    assert (dict_ < 0).any() and not np.allclose(dict_.reshape(D, k, k), dict_.reshape(D, k, k)[:, ::-1, ::-1])
    tol = tol_for(coef)
    dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
    got = host(sr.sr_dict_regress_dense(dlr, dco, ddi, r, k))
    assert max_abs_err(got, oracle.dict_regress_dense(lr, coef, dict_, r, k)) <= tol
    want = oracle.dict_regress_selected(lr, coef, None, None, dict_, r, k, s)
    got = host(sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s))
    assert max_abs_err(got, want) <= tol
    idx, sel = sr.sr_dict_select(dco, s, want_sel=True)
    got = host(sr.sr_dict_regress_selected(dlr, dco, idx, None, ddi, r, k, s))
    assert max_abs_err(got, want) <= tol
    got = host(sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, s, sr.SR_COEF_COMPACT))
    assert max_abs_err(got, want) <= tol
    rng = np.random.default_rng(5)
    S = rng.choice(D, size=s, replace=False).astype(np.uint8)
    S[0] = 1 if 1 not in S[1:] else S[0]                     # the off-centre delta atom is in the subset
    gamma = signed_gamma(s)
    assert (gamma < 0).any()
    want = oracle.dict_regress_selected(lr, coef, S, gamma, dict_, r, k, s, flags=oracle.IDX_GLOBAL)
    got = host(sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, s, sr.SR_IDX_GLOBAL))
    assert max_abs_err(got, want) <= tol
    compact = dev(coef[:, S.astype(int)].copy())
    got = host(sr.sr_dict_regress_selected(dlr, compact, dev(S), dev(gamma), ddi, r, k, s, sr.SR_IDX_GLOBAL | sr.SR_COEF_COMPACT))
    assert max_abs_err(got, want) <= tol
    assert sr.sr_device_status() == 0


@pytest.mark.parametrize("dt,w", [("f16", 48), ("f32", 48), ("f16", 35)])
@pytest.mark.parametrize("tap", [(0, 1), (4, 0), (3, 4), (2, 2)])
def test_off_centre_delta_atom_shifts_the_upsampled_image(dt, w, tap):
    """One atom that is a single tap at (a, b), one-hot coefficients: the output is the up-sampled image read at
    (Y + a - p, X + b - p), clamped to the frame. The expected frame is built from the bicubic oracle by indexing
    alone, so the pairing of taps and patch positions is checked without the oracle's own regression."""
    a, b = tap
    r, k, D, p = 4, 5, 72, 2
    wl = _wl(1, 3, 20, w, r, D, k, dt)
    lr, dict_, _ = sr_inputs.make_inputs(wl)
    dict_[3] = 0
    dict_[3, a * k + b] = 1
    coef = np.zeros((1, D, wl.H, wl.W), np.float16 if dt == "f16" else np.float32)
    coef[:, 3] = 1
    U = oracle.bicubic_upsample(lr, r)
    yy = np.clip(np.arange(wl.H) + a - p, 0, wl.H - 1)
    xx = np.clip(np.arange(wl.W) + b - p, 0, wl.W - 1)
    want = U[:, :, yy][:, :, :, xx]
    dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
    assert max_abs_err(host(sr.sr_dict_regress_dense(dlr, dco, ddi, r, k)), want) <= 2e-6
    assert max_abs_err(host(sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, 3)), want) <= 2e-6
    S = np.array([0, 3, 5], np.uint8)
    assert max_abs_err(host(sr.sr_dict_regress_selected(dlr, dco, dev(S), None, ddi, r, k, 3, sr.SR_IDX_GLOBAL)), want) <= 2e-6
    idx, sel = sr.sr_dict_select(dco, 3, want_sel=True)
    assert max_abs_err(host(sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, 3, sr.SR_COEF_COMPACT)), want) <= 2e-6
    np.testing.assert_allclose(oracle.dict_regress_dense(lr, coef, dict_, r, k), want, rtol=0, atol=1e-12)


@pytest.mark.parametrize("scale,bound", [(2.0 ** 15, TOL_F16 * 2.0 ** 15), (2.0 ** -10, 1e-5)])
def test_dictionary_magnitude_range_of_the_tensor_core_path(scale, bound):
    """The tensor-core path keeps the fp32 dictionary as a binary16 hi + lo pair, so its taps must stay below the
    largest binary16 number (65504); taps below 2^-14 fall into the binary16 subnormals and keep an absolute, not a
    relative, precision (2^-25 per tap). A large dictionary (taps up to about 9500) must be as accurate relative to
    its scale as the ordinary one; a tiny one (taps around 1e-4) within the absolute bound that follows from 2^-25 per
    tap: 3 (sum of |coefficients|) x 25 taps x 1.45 (|U|) x 2^-25 = 3.3e-6."""
    wl = _wl(1, 3, 24, 64, 2, 72, 5, "f16")
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    dict_ = (signed_asymmetric_dictionary(dict_) * np.float32(scale)).astype(np.float32)
    assert np.abs(dict_).max() < 65504
    got = host(sr.sr_dict_regress_dense(dev(lr), dev(coef), dev(dict_), 2, 5))
    assert max_abs_err(got, oracle.dict_regress_dense(lr, coef, dict_, 2, 5)) <= bound
    got = host(sr.sr_dict_regress_selected(dev(lr), dev(coef), None, None, dev(dict_), 2, 5, 8))
    assert max_abs_err(got, oracle.dict_regress_selected(lr, coef, None, None, dict_, 2, 5, 8)) <= bound
