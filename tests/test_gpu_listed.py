"""Regression from index + value planes on the gather kernel (FMA pipe), element by element against the oracle.

Two kernels serve this call: the gather kernel and the first tensor-core layout; the host rules pick by shape. The
test hook sr_test_force_kernel pins each in turn, so that both are checked on the same inputs whatever the rules
say, and the two are compared with one another as well (same lists, same fp32 accumulation: they differ only in
rounding order). Shapes span several tiles in both directions, ragged right and bottom edges, widths that are odd
multiples of two, every supported k and c, lists of 1 to 16 atoms, out-of-range indices and every output type.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, dev, host, max_abs_err, signed_asymmetric_dictionary

pytestmark = pytest.mark.gpu

GATHER, FIRST = 4, 1


@pytest.fixture(autouse=True)
def _back_to_the_host_rules():
    yield
    sr.sr_test_force_kernel(-1)


def _lists(wl, s, seed=3):
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    dict_ = signed_asymmetric_dictionary(dict_)
    idx, sel = oracle.dict_select(coef, s, want_sel=True)
    return lr, dict_, idx, sel.astype(np.float16)      # the kept values are binary16 inputs: exact


def _launches_of(fn):
    before = sr.sr_launch_count()
    out = fn()
    return out, sr.sr_launch_count() - before


@pytest.mark.parametrize("h,w,r,D,k,c,s", [
    (40, 72, 2, 72, 5, 3, 8),      # 80 x 144: a full tile column and a ragged one, several tile rows
    (23, 36, 4, 72, 5, 3, 8),      # 92 x 144, scale 4
    (30, 48, 3, 32, 3, 3, 16),     # 90 x 144, scale 3, the longest lists
    (20, 37, 2, 16, 7, 3, 4),      # 40 x 74, 7 x 7 atoms (one pixel's filter at a time); width not a multiple of 16:
                                   # the tensor-core layout does not take it and the general kernel is the other side
    (16, 64, 2, 128, 5, 1, 5),     # one channel, 128 atoms, an odd list length
    (9, 11, 2, 24, 3, 1, 1),       # a single listed atom, an image smaller than a tile
])
def test_gather_kernel_matches_the_oracle_and_the_tensor_core_layout(h, w, r, D, k, c, s):
    wl = sr_inputs.Workload("t", 2, c, h, w, r, D=D, k=k, coef_dtype="f16")
    lr, dict_, idx, sel = _lists(wl, s)
    want = oracle.dict_regress_selected(lr, sel, idx, None, dict_, r, k, s, flags=oracle.COEF_COMPACT)
    args = (dev(lr), dev(sel), dev(idx), None, dev(dict_), r, k, s, sr.SR_COEF_COMPACT)
    sr.sr_test_force_kernel(GATHER)
    got, launches = _launches_of(lambda: host(sr.sr_dict_regress_selected(*args)))
    assert launches == 1
    assert max_abs_err(got, want) <= TOL_F16
    sr.sr_test_force_kernel(FIRST)
    other = host(sr.sr_dict_regress_selected(*args))
    assert max_abs_err(other, want) <= TOL_F16
    assert np.abs(got - other).max() <= 2e-4      # both accumulate in fp32; only the order of the sums differs
    assert sr.sr_device_status() == 0


def test_the_search_times_the_gather_kernel_too():
    wl = sr_inputs.Workload("t", 1, 3, 48, 64, 2, D=72, k=3, coef_dtype="f16")
    lr, dict_, idx, sel = _lists(wl, 4)
    args = (dev(lr), dev(sel), dev(idx), None, dev(dict_), 2, 3, 4, sr.SR_COEF_COMPACT)
    res = sr.sr_tune_selected(*args, reps=3)
    sr.sr_tune_reset()
    assert res["candidates"] >= 4                      # the first layout and the gather kernel's three tile heights
    assert res["kernel"] in ("gather (FMA pipe)", "first tensor-core layout")
    assert res["best_us"] <= res["default_us"] * 1.0001


def test_indices_beyond_the_dictionary_read_its_last_atom():
    wl = sr_inputs.Workload("t", 1, 3, 16, 32, 2, D=20, k=5, coef_dtype="f16")
    lr, dict_, idx, sel = _lists(wl, 4)
    bad = idx.copy()
    bad[:, 1, ::3, ::5] = 200                          # listed atom does not exist: both sides clamp to atom D - 1
    clamped = np.minimum(bad, 19).astype(np.uint8)
    want = oracle.dict_regress_selected(lr, sel, clamped, None, dict_, 2, 5, 4, flags=oracle.COEF_COMPACT)
    sr.sr_test_force_kernel(GATHER)
    got = host(sr.sr_dict_regress_selected(dev(lr), dev(sel), dev(bad), None, dev(dict_), 2, 5, 4, sr.SR_COEF_COMPACT))
    assert max_abs_err(got, want) <= TOL_F16


@pytest.mark.parametrize("flag,dtype", [(sr.SR_OUT_F16, torch.float16), (sr.SR_OUT_U8, torch.uint8)])
def test_output_types_and_clamp(flag, dtype):
    wl = sr_inputs.Workload("t", 1, 3, 24, 40, 4, D=72, k=5, coef_dtype="f16")
    lr, dict_, idx, sel = _lists(wl, 8)
    dict_ = (dict_ * 1.5).astype(np.float32)           # pushes values outside [0, 1]: the clamp has work to do
    want = oracle.dict_regress_selected(lr, sel, idx, None, dict_, 4, 5, 8, flags=oracle.COEF_COMPACT | oracle.CLAMP01)
    sr.sr_test_force_kernel(GATHER)
    got = sr.sr_dict_regress_selected(dev(lr), dev(sel), dev(idx), None, dev(dict_), 4, 5, 8,
                                      sr.SR_COEF_COMPACT | sr.SR_CLAMP01 | flag)
    assert got.dtype == dtype
    if dtype == torch.uint8:
        assert np.abs(host(got).astype(np.int32) - np.rint(want * 255.0).astype(np.int32)).max() <= 1
    else:
        assert max_abs_err(host(got).astype(np.float32), want) <= TOL_F16 + 1e-3      # binary16 rounding of the result


def test_full_frame_sampled_against_the_oracle():
    """The bench configuration (1080p x4, D = 72, k = 5, s = 8), where the host rules keep the tensor-core layout, on
    the gather kernel: compared with the oracle on sampled pixels (seeded random set, corners, both sides of tile
    seams) and with the tensor-core layout on every pixel."""
    wl = sr_inputs.CONFIGS["cfg1"]
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    dlr, ddi, dco = dev(lr), dev(dict_), dev(coef)
    idx, sel = sr.sr_dict_select(dco, wl.s, want_sel=True)
    del dco
    fl = sr.SR_COEF_COMPACT | sr.SR_CLAMP01
    sr.sr_test_force_kernel(GATHER)
    got = sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, wl.scale, wl.k, wl.s, fl)
    sr.sr_test_force_kernel(FIRST)
    other = sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, wl.scale, wl.k, wl.s, fl)
    assert float((got - other).abs().max()) <= 2e-4
    rng = np.random.default_rng(5)
    H, W = wl.H, wl.W
    ys = np.concatenate([[0, 1, H - 2, H - 1], np.arange(7, H, 8)[:40], np.arange(8, H, 8)[:40]])
    xs = np.concatenate([[0, 1, 63, 64, 127, 128, W - 2, W - 1], rng.integers(0, W, 24)])
    samples = np.unique(np.concatenate([(ys[:, None] * W + xs[None, :]).ravel(), rng.integers(0, H * W, 20000)]).astype(np.int64))
    want = oracle.regress_at("selected", lr, coef, None, None, dict_, samples, wl.scale, wl.k, s=wl.s, flags=oracle.CLAMP01)
    flat = got.reshape(1, 3, -1)[0][:, torch.from_numpy(samples).cuda()].T.cpu().numpy()
    assert max_abs_err(flat, want) <= TOL_F16
    assert sr.sr_device_status() == 0
