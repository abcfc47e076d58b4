"""SR_OUT_F16: the regression calls store their fp32 result rounded to binary16.  Every mode against the oracle on
shapes that reach the tensor-core kernels and the general kernel; the bound is the path's own tolerance plus half a
binary16 unit in the last place of the exact value, and the stored values equal the fp32 output rounded to nearest.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, TOL_F32, dev, host

pytestmark = pytest.mark.gpu

H16 = sr.SR_OUT_F16
CASES = [
    ("tensor_th16", 1, 3, 24, 40, 4, 72, 5, "f16", 8),
    ("tensor_k3_c2", 2, 2, 30, 32, 2, 32, 3, "f16", 4),
    ("tensor_k7", 1, 3, 16, 48, 3, 24, 7, "f16", 12),
    ("short_last_tile", 1, 3, 13, 32, 3, 16, 5, "f16", 4),     # 39 rows: 16 + 16 + 7
    ("fma_f32", 1, 3, 17, 19, 2, 16, 5, "f32", 4),
]


def _check(got16, want, tol):
    assert got16.dtype == np.float16
    bound = tol + np.abs(want) * 2.0 ** -11 + 2.0 ** -25        # half an ulp of binary16 (normal range), subnormal floor
    err = np.abs(got16.astype(np.float64) - want)
    assert np.all(err <= bound), float(np.max(err - bound))


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_all_modes_store_binary16(case):
    name, n, c, h, w, r, D, k, dt, s = case
    wl = sr_inputs.Workload(name, n, c, h, w, r, D, k, dt, s)
    lr, dict_, coef = sr_inputs.make_inputs(wl, seed=91)
    tol = TOL_F16 if dt == "f16" else TOL_F32
    dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
    want = oracle.dict_regress_dense(lr, coef, dict_, r, k)
    got32 = sr.sr_dict_regress_dense(dlr, dco, ddi, r, k, 0)
    got16 = sr.sr_dict_regress_dense(dlr, dco, ddi, r, k, H16)
    _check(host(got16), want, tol)
    assert torch.equal(got16, got32.to(torch.float16))          # the same fp32 value, rounded to nearest even
    want_s = oracle.dict_regress_selected(lr, coef, None, None, dict_, r, k, s, flags=oracle.CLAMP01)
    fl = H16 | sr.SR_CLAMP01
    _check(host(sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s, fl)), want_s, tol)
    idx, sel = sr.sr_dict_select(dco, s, want_sel=True)
    _check(host(sr.sr_dict_regress_selected(dlr, dco, idx, None, ddi, r, k, s, fl)), want_s, tol)
    _check(host(sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, s, fl | sr.SR_COEF_COMPACT)), want_s, tol)
    S = np.arange(0, D, max(1, D // s), dtype=np.uint8)[:s]
    gamma = np.linspace(0.75, 1.25, S.size).astype(np.float32)
    want_g = oracle.dict_regress_selected(lr, coef, S, gamma, dict_, r, k, S.size, flags=oracle.IDX_GLOBAL | oracle.CLAMP01)
    got = sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, S.size, fl | sr.SR_IDX_GLOBAL)
    _check(host(got), want_g, tol)
    assert sr.sr_device_status() == 0


def test_binding_checks_the_output_type():
    wl = sr_inputs.Workload("t", 1, 3, 8, 8, 2, 8, 3, "f16", 2)
    lr, dict_, coef = sr_inputs.make_inputs(wl, seed=1)
    out32 = torch.empty((1, 3, 16, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(TypeError):
        sr.sr_dict_regress_dense(dev(lr), dev(coef), dev(dict_), 2, 3, H16, out=out32)
