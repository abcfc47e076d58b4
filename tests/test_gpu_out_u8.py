"""SR_OUT_U8: the regression calls store an 8-bit image, code = round-to-nearest-even(255 * clamp(value, 0, 1)).

The rounding decision is taken in the kernel's precision (fp32), so the codes must be bit-equal to the same call's fp32
output quantised the same way; against the fp64 oracle's codes they may differ by one where the fp32 value sits within
the path's tolerance of a rounding boundary, and nowhere else. Every mode, on shapes that reach each kernel (both
tensor-core layouts, the FMA-pipe subset kernel, the general kernel).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, TOL_F32, dev, host

pytestmark = pytest.mark.gpu

U8 = sr.SR_OUT_U8
CASES = [
    ("first_layout", 1, 3, 24, 40, 4, 72, 5, "f16", 8),
    ("second_layout_few_atoms", 2, 3, 30, 32, 2, 16, 3, "f16", 12),
    ("second_layout_k7", 1, 3, 16, 48, 3, 24, 7, "f16", 12),
    ("short_last_tile", 1, 3, 13, 32, 3, 16, 5, "f16", 4),
    ("general_f32", 1, 3, 17, 19, 2, 16, 5, "f32", 4),
    ("one_channel", 1, 1, 20, 32, 2, 40, 5, "f16", 8),
]


def _quantise_f32(t: torch.Tensor) -> torch.Tensor:
    """The kernel's own rule on its own fp32 value: clamp, times 255 in fp32, round half to even."""
    return torch.round(torch.clamp(t, 0.0, 1.0) * 255.0).to(torch.uint8)


def _check_against_oracle(codes: np.ndarray, want_value: np.ndarray, want_codes: np.ndarray, tol: float):
    assert codes.dtype == np.uint8
    diff = codes.astype(np.int64) - want_codes.astype(np.int64)
    assert np.abs(diff).max() <= 1
    scaled = 255.0 * np.clip(want_value, 0.0, 1.0)
    near_boundary = np.abs(scaled - np.floor(scaled) - 0.5) <= 255.0 * tol
    assert not np.any((diff != 0) & ~near_boundary)          # a different code only where fp32 may round the other way


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_all_modes_store_eight_bit_codes(case):
    name, n, c, h, w, r, D, k, dt, s = case
    wl = sr_inputs.Workload(name, n, c, h, w, r, D, k, dt, s)
    lr, dict_, coef = sr_inputs.make_inputs(wl, seed=77)
    tol = TOL_F16 if dt == "f16" else TOL_F32
    dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
    idx, sel = sr.sr_dict_select(dco, s, want_sel=True)
    S = np.arange(0, D, max(1, D // s), dtype=np.uint8)[:s]
    gamma = np.linspace(0.75, 1.25, S.size).astype(np.float32)
    calls = {
        "dense": (lambda fl: sr.sr_dict_regress_dense(dlr, dco, ddi, r, k, fl),
                  lambda fl: oracle.dict_regress_dense(lr, coef, dict_, r, k, flags=fl)),
        "fused": (lambda fl: sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s, fl),
                  lambda fl: oracle.dict_regress_selected(lr, coef, None, None, dict_, r, k, s, flags=fl)),
        "index_planes": (lambda fl: sr.sr_dict_regress_selected(dlr, dco, idx, None, ddi, r, k, s, fl),
                         lambda fl: oracle.dict_regress_selected(lr, coef, None, None, dict_, r, k, s, flags=fl)),
        "compact": (lambda fl: sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, s, fl | sr.SR_COEF_COMPACT),
                    lambda fl: oracle.dict_regress_selected(lr, coef, None, None, dict_, r, k, s, flags=fl)),
        "global": (lambda fl: sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, S.size, fl | sr.SR_IDX_GLOBAL),
                   lambda fl: oracle.dict_regress_selected(lr, coef, S, gamma, dict_, r, k, S.size, flags=fl | oracle.IDX_GLOBAL)),
    }
    for mode, (gpu, ref) in calls.items():
        codes = gpu(U8)
        assert codes.dtype == torch.uint8, mode
        assert torch.equal(codes, _quantise_f32(gpu(0))), mode              # same fp32 value, same rounding rule
        assert torch.equal(codes, gpu(U8 | sr.SR_CLAMP01)), mode            # the clamp is implied
        _check_against_oracle(host(codes), ref(0), ref(oracle.OUT_U8), tol)
    assert sr.sr_device_status() == 0


def test_eight_bit_and_binary16_output_exclude_each_other():
    wl = sr_inputs.Workload("t", 1, 3, 8, 8, 2, 8, 3, "f16", 2)
    lr, dict_, coef = sr_inputs.make_inputs(wl, seed=1)
    with pytest.raises(sr.SrError) as e:
        sr.sr_dict_regress_dense(dev(lr), dev(coef), dev(dict_), 2, 3, U8 | sr.SR_OUT_F16)
    assert e.value.status == sr.api.SR_ERR_UNSUPPORTED
    out32 = torch.empty((1, 3, 16, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(TypeError):
        sr.sr_dict_regress_dense(dev(lr), dev(coef), dev(dict_), 2, 3, U8, out=out32)
