"""SR_LUMA_ONLY: the per-pixel filter acts on the BT.601 luma of the up-sampled image, the chroma differences keep
their up-sampled values. Every mode against the oracle, with each output type, on shapes that the other kernels would
otherwise take (the flag has to route them to the general kernel) and with both stage-1 interpolations.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, TOL_F32, dev, host, signed_asymmetric_dictionary, signed_gamma

pytestmark = pytest.mark.gpu

LU = sr.SR_LUMA_ONLY
CASES = [
    ("first_layout_shape", 1, 24, 40, 4, 72, 5, "f16", 8),
    ("second_layout_shape", 2, 30, 32, 2, 16, 3, "f16", 12),
    ("subset_kernel_shape", 1, 16, 48, 3, 24, 7, "f16", 8),
    ("ragged_f32", 1, 17, 19, 2, 16, 5, "f32", 4),
    ("k9_r1", 1, 33, 37, 1, 12, 9, "f16", 3),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_every_mode_matches_the_oracle(case):
    name, n, h, w, r, D, k, dt, s = case
    wl = sr_inputs.Workload(name, n, 3, h, w, r, D, k, dt, s)
    lr, dict_, coef = sr_inputs.make_inputs(wl, seed=5)
    dict_ = signed_asymmetric_dictionary(dict_)
    tol = TOL_F16 if dt == "f16" else TOL_F32
    dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
    idx, sel = sr.sr_dict_select(dco, s, want_sel=True)
    S = np.arange(0, D, max(1, D // s), dtype=np.uint8)[:s]
    gamma = signed_gamma(S.size)
    for up, oup in ((0, 0), (sr.SR_UPSAMPLE_BILINEAR, oracle.UPSAMPLE_BILINEAR)):
        fl, ofl = LU | sr.SR_CLAMP01 | up, oracle.LUMA_ONLY | oracle.CLAMP01 | oup
        want = oracle.dict_regress_dense(lr, coef, dict_, r, k, flags=ofl)
        got = sr.sr_dict_regress_dense(dlr, dco, ddi, r, k, fl)
        assert np.abs(host(got) - want).max() <= tol
        # not the ordinary regression by another name: the two differ on a colour image
        assert np.abs(want - oracle.dict_regress_dense(lr, coef, dict_, r, k, flags=ofl & ~oracle.LUMA_ONLY)).max() > 100 * tol
        want = oracle.dict_regress_selected(lr, coef, None, None, dict_, r, k, s, flags=ofl)
        for got in (sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s, fl),
                    sr.sr_dict_regress_selected(dlr, dco, idx, None, ddi, r, k, s, fl),
                    sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, s, fl | sr.SR_COEF_COMPACT)):
            assert np.abs(host(got) - want).max() <= tol
        want = oracle.dict_regress_selected(lr, coef, S, gamma, dict_, r, k, S.size, flags=ofl | oracle.IDX_GLOBAL)
        got = sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, S.size, fl | sr.SR_IDX_GLOBAL)
        assert np.abs(host(got) - want).max() <= tol
    assert sr.sr_device_status() == 0


def test_output_types_and_chroma():
    wl = sr_inputs.Workload("t", 1, 3, 20, 32, 2, 40, 5, "f16", 8)
    lr, dict_, coef = sr_inputs.make_inputs(wl, seed=9)
    dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
    f32 = sr.sr_dict_regress_dense(dlr, dco, ddi, 2, 5, LU)
    f16 = sr.sr_dict_regress_dense(dlr, dco, ddi, 2, 5, LU | sr.SR_OUT_F16)
    u8 = sr.sr_dict_regress_dense(dlr, dco, ddi, 2, 5, LU | sr.SR_OUT_U8)
    # the fp32 form is composed of the fast one-channel regression and two small kernels, the other output types run on
    # the general kernel: same definition, different rounding order
    assert f16.dtype == torch.float16 and float((f16.float() - f32).abs().max()) <= 2 * TOL_F16 + 1e-3
    codes = torch.round(torch.clamp(f32, 0, 1) * 255).to(torch.int16)
    assert u8.dtype == torch.uint8 and int((u8.to(torch.int16) - codes).abs().max()) <= 1
    # without a clamp every channel moves by the same amount: differences between channels are those of stage 1
    U = sr.sr_bicubic_upsample(dlr, 2)
    assert float(((f32[:, 0] - f32[:, 1]) - (U[:, 0] - U[:, 1])).abs().max()) <= 1e-6
    assert float(((f32[:, 2] - f32[:, 1]) - (U[:, 2] - U[:, 1])).abs().max()) <= 1e-6


def test_needs_three_channels():
    wl = sr_inputs.Workload("t", 1, 1, 8, 8, 2, 8, 3, "f16", 4)
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    with pytest.raises(sr.SrError):
        sr.sr_dict_regress_dense(dev(lr), dev(coef), dev(dict_), 2, 3, LU)
