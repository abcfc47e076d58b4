"""Seeded random small shapes through every entry point and mode, element by element against the oracle.

The fixed parity cases pick shapes by hand; this sweep draws them (scale, patch size, channels, batch, atom count,
atoms kept, ragged heights, HR widths that are multiples of 8 or 16, inputs with and without exact magnitude ties)
so that combinations nobody thought of are still exercised: tile seams, partial 8-atom groups, both tile heights,
the tensor-core and the general kernels.
"""
import numpy as np
import pytest

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, dev, host, signed_asymmetric_dictionary

pytestmark = pytest.mark.gpu


def _draw(rng):
    r = int(rng.choice([1, 2, 3, 4]))
    k = int(rng.choice([3, 5, 7]))
    c = int(rng.choice([1, 2, 3, 4]))
    n = int(rng.choice([1, 1, 2]))
    D = int(rng.choice([6, 8, 16, 20, 24, 32, 40, 72, 100, 128]))
    s = int(min(D, rng.choice([1, 2, 3, 4, 5, 8, 9, 12, 16])))
    W = int(rng.choice([8, 16, 16])) * int(rng.integers(1, 20))
    H = int(rng.integers(3, 70))
    if W % r or H % r:
        W, H = W * r, H * r
    return sr_inputs.Workload("random", n, c, H // r, W // r, r, D, k, "f16", s)


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_shapes_all_modes(seed):
    rng = np.random.default_rng(seed)
    for case in range(16):
        wl = _draw(rng)
        r, k, s, D = wl.scale, wl.k, wl.s, wl.D
        lr, dict_, coef = sr_inputs.make_inputs(wl, seed=1000 * seed + case)
        if rng.random() < 0.4:   # coarse grid: exact magnitude ties, +/- pairs and zeros are frequent
            coef = (np.round(coef.astype(np.float32) * 64) / 64).astype(coef.dtype)
        if case % 2:             # every second case: atoms without symmetry and with both signs
            dict_ = signed_asymmetric_dictionary(dict_, seed=case)
        tag = f"seed {seed} case {case}: {wl}"
        dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
        err = np.abs(host(sr.sr_bicubic_upsample(dlr, r)).astype(np.float64) - oracle.bicubic_upsample(lr, r)).max()
        assert err <= 2e-6, tag
        err = np.abs(host(sr.sr_dict_regress_dense(dlr, dco, ddi, r, k)) - oracle.dict_regress_dense(lr, coef, dict_, r, k)).max()
        assert err <= TOL_F16, tag
        want = oracle.dict_regress_selected(lr, coef, None, None, dict_, r, k, s)
        err = np.abs(host(sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s)) - want).max()
        assert err <= TOL_F16, tag
        idx, sel = sr.sr_dict_select(dco, s, want_sel=True)
        np.testing.assert_array_equal(host(idx), oracle.dict_select(coef, s), err_msg=tag)
        err = np.abs(host(sr.sr_dict_regress_selected(dlr, dco, idx, None, ddi, r, k, s)) - want).max()
        assert err <= TOL_F16, tag
        err = np.abs(host(sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, s, sr.SR_COEF_COMPACT)) - want).max()
        assert err <= TOL_F16, tag
        S = rng.choice(D, size=s, replace=False).astype(np.uint8)
        gamma = (rng.uniform(0.5, 1.5, size=s) * rng.choice([-1.0, 1.0], size=s)).astype(np.float32)
        want = oracle.dict_regress_selected(lr, coef, S, gamma, dict_, r, k, s, flags=oracle.IDX_GLOBAL)
        err = np.abs(host(sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, s, sr.SR_IDX_GLOBAL)) - want).max()
        assert err <= TOL_F16, tag
        assert sr.sr_device_status() == 0, tag


def _draw_wide(rng):
    """Wider draw than _draw: k in {1, 9}, up to 200 atoms, s beyond the tensor path's 16, fp32 coefficients, HR widths
    that are only multiples of 4 (general kernel)."""
    r = int(rng.choice([1, 2, 3, 4, 5]))
    k = int(rng.choice([1, 3, 5, 7, 9]))
    c = int(rng.choice([1, 2, 3, 4]))
    n = int(rng.choice([1, 1, 2]))
    D = int(rng.choice([6, 8, 16, 20, 24, 32, 40, 72, 100, 128, 200]))
    s = int(min(D, rng.choice([1, 2, 3, 4, 5, 8, 9, 12, 16, 20])))
    W = int(rng.choice([8, 16, 16, 4])) * int(rng.integers(1, 20))
    H = int(rng.integers(3, 70))
    if W % r or H % r:
        W, H = W * r, H * r
    dt = "f16" if rng.random() < 0.8 else "f32"
    return sr_inputs.Workload("random", n, c, H // r, W // r, r, D, k, dt, s)


@pytest.mark.parametrize("seed", [11, 12])
def test_random_shapes_random_flags(seed):
    """Every regression mode with a random combination of the output clamp, the bilinear up-sampling and binary16
    output; the bound is the path's tolerance plus, for binary16 output, half a unit in its last place."""
    rng = np.random.default_rng(seed)
    for case in range(20):
        wl = _draw_wide(rng)
        r, k, s, D = wl.scale, wl.k, wl.s, wl.D
        if k == 1:   # the dictionary generator has no 1 x 1 atoms: take the centre taps of a 3 x 3 one
            lr, dict_, coef = sr_inputs.make_inputs(sr_inputs.Workload("random", wl.n, wl.c, wl.h, wl.w, r, D, 3, wl.coef_dtype, s),
                                                    seed=3000 * seed + case)
            dict_ = np.ascontiguousarray(dict_[:, 4:5])
        else:
            lr, dict_, coef = sr_inputs.make_inputs(wl, seed=3000 * seed + case)
        if rng.random() < 0.4:
            coef = (np.round(coef.astype(np.float32) * 64) / 64).astype(coef.dtype)
        if case % 2:
            dict_ = signed_asymmetric_dictionary(dict_, seed=case)
        fl = ofl = 0
        if rng.random() < 0.5:
            fl, ofl = fl | sr.SR_CLAMP01, ofl | oracle.CLAMP01
        bilinear = rng.random() < 0.5
        if bilinear:
            fl, ofl = fl | sr.SR_UPSAMPLE_BILINEAR, ofl | oracle.UPSAMPLE_BILINEAR
        f16_out = rng.random() < 0.5
        if f16_out:
            fl |= sr.SR_OUT_F16
        tol = TOL_F16 if coef.dtype == np.float16 else 1e-5
        tag = f"seed {seed} case {case}: {wl} flags {fl}"

        def check(got, want):
            bound = tol + (np.abs(want) * 2.0 ** -11 + 2.0 ** -25 if f16_out else 0.0)
            assert np.all(np.abs(host(got).astype(np.float64) - want) <= bound), tag

        dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
        check(sr.sr_dict_regress_dense(dlr, dco, ddi, r, k, fl), oracle.dict_regress_dense(lr, coef, dict_, r, k, flags=ofl))
        want = oracle.dict_regress_selected(lr, coef, None, None, dict_, r, k, s, flags=ofl)
        check(sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s, fl), want)
        idx, sel = sr.sr_dict_select(dco, s, want_sel=True)
        np.testing.assert_array_equal(host(idx), oracle.dict_select(coef, s), err_msg=tag)
        check(sr.sr_dict_regress_selected(dlr, dco, idx, None, ddi, r, k, s, fl), want)
        check(sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, s, fl | sr.SR_COEF_COMPACT), want)
        S = rng.choice(D, size=s, replace=False).astype(np.uint8)
        gamma = (rng.uniform(0.5, 1.5, size=s) * rng.choice([-1.0, 1.0], size=s)).astype(np.float32)
        want = oracle.dict_regress_selected(lr, coef, S, gamma, dict_, r, k, s, flags=ofl | oracle.IDX_GLOBAL)
        check(sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, s, fl | sr.SR_IDX_GLOBAL), want)
        up = (sr.sr_bilinear_upsample if bilinear else sr.sr_bicubic_upsample)(dlr, r)
        want_up = (oracle.bilinear_upsample if bilinear else oracle.bicubic_upsample)(lr, r)
        assert np.abs(host(up).astype(np.float64) - want_up).max() <= 2e-6, tag
        assert sr.sr_device_status() == 0, tag
