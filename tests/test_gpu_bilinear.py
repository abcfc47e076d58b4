"""Bilinear variant of stage 1 (`sr_bilinear_upsample`, `SR_UPSAMPLE_BILINEAR`): every entry point and mode against
the oracle, element by element, on shapes that reach the tensor-core kernels (both tile heights), the general FMA
kernel and the stand-alone block / direct up-sampling kernels; plus the 1080p x4 frame on sampled pixels.
"""
import numpy as np
import pytest

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, TOL_F32, dev, host

pytestmark = pytest.mark.gpu

B = sr.SR_UPSAMPLE_BILINEAR
OB = oracle.UPSAMPLE_BILINEAR


@pytest.mark.parametrize("r,h,w,n,c", [(1, 7, 9, 1, 3), (2, 33, 40, 2, 3), (3, 20, 17, 1, 2), (4, 19, 36, 1, 3),
                                        (5, 6, 11, 1, 1), (8, 5, 4, 1, 4), (4, 1, 1, 1, 1)])
def test_upsample_alone(r, h, w, n, c):
    lr = np.random.default_rng(r * 100 + h).random((n, c, h, w), dtype=np.float32)
    got = host(sr.sr_bilinear_upsample(dev(lr), r))
    want = oracle.bilinear_upsample(lr, r)
    assert np.max(np.abs(got - want)) <= 2e-7       # two fp32 products and a sum of values in [0, 1)
    assert sr.sr_device_status() == 0


CASES = [
    # name, n, c, h, w, r, D, k, dtype, s
    ("tensor_th16", 1, 3, 24, 40, 4, 72, 5, "f16", 8),
    ("tensor_k3", 2, 3, 30, 32, 2, 32, 3, "f16", 4),
    ("tensor_k7_r3", 1, 2, 16, 48, 3, 24, 7, "f16", 12),
    ("ragged_w", 1, 3, 13, 22, 4, 20, 5, "f16", 5),
    ("fma_f32", 1, 3, 17, 19, 2, 16, 5, "f32", 4),
    ("fma_k9", 1, 1, 9, 10, 2, 8, 9, "f16", 3),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("clamp", [0, sr.SR_CLAMP01])
def test_all_modes(case, clamp):
    name, n, c, h, w, r, D, k, dt, s = case
    wl = sr_inputs.Workload(name, n, c, h, w, r, D, k, dt, s)
    lr, dict_, coef = sr_inputs.make_inputs(wl, seed=77)
    tol = TOL_F16 if dt == "f16" else TOL_F32
    dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
    fl, ofl = B | clamp, OB | (oracle.CLAMP01 if clamp else 0)
    want = oracle.dict_regress_dense(lr, coef, dict_, r, k, flags=ofl)
    assert np.max(np.abs(host(sr.sr_dict_regress_dense(dlr, dco, ddi, r, k, fl)) - want)) <= tol
    # the variant really is a different image: the bicubic result differs by more than the tolerance somewhere
    if h > 2 and w > 2 and r > 1:
        assert np.max(np.abs(oracle.dict_regress_dense(lr, coef, dict_, r, k, flags=ofl & ~OB) - want)) > 10 * tol
    want_s = oracle.dict_regress_selected(lr, coef, None, None, dict_, r, k, s, flags=ofl)
    got = host(sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s, fl))
    assert np.max(np.abs(got - want_s)) <= tol
    idx, sel = sr.sr_dict_select(dco, s, want_sel=True)
    got = host(sr.sr_dict_regress_selected(dlr, dco, idx, None, ddi, r, k, s, fl))
    assert np.max(np.abs(got - want_s)) <= tol
    got = host(sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, s, fl | sr.SR_COEF_COMPACT))
    assert np.max(np.abs(got - want_s)) <= tol
    S = np.arange(0, D, max(1, D // s), dtype=np.uint8)[:s]
    gamma = np.linspace(0.75, 1.25, S.size).astype(np.float32)
    want_g = oracle.dict_regress_selected(lr, coef, S, gamma, dict_, r, k, S.size, flags=ofl | oracle.IDX_GLOBAL)
    got = host(sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, S.size, fl | sr.SR_IDX_GLOBAL))
    assert np.max(np.abs(got - want_g)) <= tol
    assert sr.sr_device_status() == 0


def test_full_frame_sampled():
    """cfg1 (1080p x4, D = 72, k = 5, binary16): dense and fused-selective results at sampled pixels, borders included."""
    wl = [c for c in sr_inputs.CONFIGS if c.name.startswith("cfg1")][0] if not isinstance(sr_inputs.CONFIGS, dict) else sr_inputs.CONFIGS["cfg1"]
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    r, k, s = wl.scale, wl.k, wl.s
    dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
    rng = np.random.default_rng(5)
    HW = wl.H * wl.W
    samples = np.unique(np.concatenate([rng.integers(0, HW, 600), np.arange(0, 64), np.arange(HW - 64, HW),
                                        np.arange(0, HW, wl.W)[:40], np.arange(wl.W - 1, HW, wl.W)[:40]])).astype(np.int64)
    dense = host(sr.sr_dict_regress_dense(dlr, dco, ddi, r, k, B)).reshape(wl.c, HW)
    want = oracle.regress_at("dense", lr, coef, None, None, dict_, samples, r, k, flags=OB)
    assert np.max(np.abs(dense[:, samples].T - want.reshape(samples.size, wl.c))) <= TOL_F16
    fused = host(sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s, B)).reshape(wl.c, HW)
    want = oracle.regress_at("fused", lr, coef, None, None, dict_, samples, r, k, s=s, flags=OB)
    assert np.max(np.abs(fused[:, samples].T - want.reshape(samples.size, wl.c))) <= TOL_F16
    up = host(sr.sr_bilinear_upsample(dlr, r))
    assert np.max(np.abs(up - oracle.bilinear_upsample(lr, r))) <= 2e-7
    assert sr.sr_device_status() == 0
