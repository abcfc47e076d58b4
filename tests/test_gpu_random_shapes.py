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
from gpu_util import TOL_F16, dev, host

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
        gamma = rng.uniform(0.5, 1.5, size=s).astype(np.float32)
        want = oracle.dict_regress_selected(lr, coef, S, gamma, dict_, r, k, s, flags=oracle.IDX_GLOBAL)
        err = np.abs(host(sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, s, sr.SR_IDX_GLOBAL)) - want).max()
        assert err <= TOL_F16, tag
        assert sr.sr_device_status() == 0, tag
