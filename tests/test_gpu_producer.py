"""Regression fused with the producer of Phi (last convolution + pixel-shuffle) against the oracle, through the C ABI.

The fused kernel never forms the coefficient tensor: it convolves the LR feature map with weights folded with the
dictionary on the tensor cores and filters the up-sampled image in its epilogue. The oracle forms Phi in fp64 from
the same features, weights and bias, then applies the definition. Tolerance: the folded weights are rounded to
binary16 (as stored coefficients would have been), so the binary16 tolerance of the other paths applies; the
observed error is far below it and a tighter bound derived from the weights' rounding is asserted as well.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, dev, host, signed_asymmetric_dictionary, signed_gamma

pytestmark = pytest.mark.gpu

TIGHT = 6e-4   # ~25 taps x (288-term dot product with weights rounded to 11 bits), see the docstring

#        name                    n  c  h   w   r  D   k  kc
CASES = [("r4_k5_ragged",        1, 3, 12, 40, 4, 8,  5, 3),
         ("r4_k5_two_frames",    2, 3, 9,  33, 4, 24, 5, 3),
         ("r4_k3",               1, 3, 8,  32, 4, 16, 3, 3),
         ("r4_k7",               1, 3, 10, 36, 4, 12, 7, 3),
         ("r4_k5_1x1",           1, 3, 7,  35, 4, 16, 5, 1),
         ("r2_k5",               1, 3, 10, 70, 2, 16, 5, 3),
         ("r2_k3_one_channel",   1, 1, 5,  64, 2, 8,  3, 3),
         ("r2_k7",               2, 2, 6,  66, 2, 10, 7, 1),
         ("r4_k5_many_tiles",    1, 3, 40, 72, 4, 72, 5, 3),
         ("r3_k5_ragged",        1, 3, 11, 50, 3, 16, 5, 3),
         ("r3_k3_two_frames",    2, 3, 7,  90, 3, 12, 3, 1),
         ("r3_k5_one_channel",   1, 1, 20, 42, 3, 72, 5, 3)]


def _make(case, seed=21):
    name, n, c, h, w, r, D, k, kc = case
    wl = sr_inputs.Workload(name, n, c, h, w, r, D=D, k=k)
    lr, dict_, _ = sr_inputs.make_inputs(wl, seed=seed)
    dict_ = signed_asymmetric_dictionary(dict_)
    feat, wconv, bias = sr_inputs.make_producer(wl, cin=32, kc=kc, seed=seed)
    return wl, lr, dict_, feat, wconv, bias


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_dense_matches_the_oracle(case):
    wl, lr, dict_, feat, wconv, bias = _make(case)
    r, k, kc = wl.scale, wl.k, wconv.shape[2]
    folded = sr.sr_producer_fold(dev(wconv), dev(bias), dev(dict_), r, k)
    got = sr.sr_producer_regress(dev(lr), torch.from_numpy(feat).cuda(), folded, r, k, wl.D, kc)
    want = oracle.producer_regress(lr, feat, wconv, bias, dict_, r, k)
    err = np.abs(host(got) - want).max()
    assert err <= TIGHT and err <= TOL_F16, err
    assert sr.sr_device_status() == 0
    # with the clamp, and a second call on the same folded block (nothing in it is consumed)
    got = sr.sr_producer_regress(dev(lr), torch.from_numpy(feat).cuda(), folded, r, k, wl.D, kc, sr.SR_CLAMP01)
    want = oracle.producer_regress(lr, feat, wconv, bias, dict_, r, k, flags=oracle.CLAMP01)
    assert np.abs(host(got) - want).max() <= TIGHT


def test_equals_the_dense_call_on_the_tensor_the_producer_would_have_stored():
    """Same result (within both paths' tolerances) as materialising Phi in binary16 and calling the dense regression."""
    wl, lr, dict_, feat, wconv, bias = _make(CASES[0])
    phi16 = sr_inputs.round_f16(oracle.producer_coef(feat, wconv, bias, wl.scale).astype(np.float32))
    dense = sr.sr_dict_regress_dense(dev(lr), torch.from_numpy(phi16).cuda(), dev(dict_), wl.scale, wl.k)
    folded = sr.sr_producer_fold(dev(wconv), dev(bias), dev(dict_), wl.scale, wl.k)
    fused = sr.sr_producer_regress(dev(lr), torch.from_numpy(feat).cuda(), folded, wl.scale, wl.k, wl.D, 3)
    assert float((dense - fused).abs().max()) <= 2 * TOL_F16


def test_subset_fold_bias_free_bilinear_and_output_types():
    wl, lr, dict_, feat, wconv, bias = _make(CASES[1])
    r, k = wl.scale, wl.k
    dlr, dfe = dev(lr), torch.from_numpy(feat).cuda()
    S = np.array([3, 17, 0, 9, 22], dtype=np.uint8)
    gamma = signed_gamma(S.size)
    folded = sr.sr_producer_fold(dev(wconv), dev(bias), dev(dict_), r, k, idx=dev(S), gamma=dev(gamma))
    got = sr.sr_producer_regress(dlr, dfe, folded, r, k, wl.D, 3)
    want = oracle.producer_regress(lr, feat, wconv, bias, dict_, r, k, idx=S, gamma=gamma)
    assert np.abs(host(got) - want).max() <= TIGHT
    folded = sr.sr_producer_fold(dev(wconv), None, dev(dict_), r, k)
    got = sr.sr_producer_regress(dlr, dfe, folded, r, k, wl.D, 3, sr.SR_UPSAMPLE_BILINEAR)
    want = oracle.producer_regress(lr, feat, wconv, None, dict_, r, k, flags=oracle.UPSAMPLE_BILINEAR)
    assert np.abs(host(got) - want).max() <= TIGHT
    folded = sr.sr_producer_fold(dev(wconv), dev(bias), dev(dict_), r, k)
    f32 = sr.sr_producer_regress(dlr, dfe, folded, r, k, wl.D, 3)
    f16 = sr.sr_producer_regress(dlr, dfe, folded, r, k, wl.D, 3, sr.SR_OUT_F16)
    u8 = sr.sr_producer_regress(dlr, dfe, folded, r, k, wl.D, 3, sr.SR_OUT_U8)
    assert f16.dtype == torch.float16 and torch.equal(f16, f32.to(torch.float16))
    assert u8.dtype == torch.uint8 and torch.equal(u8, torch.round(torch.clamp(f32, 0, 1) * 255).to(torch.uint8))
    assert sr.sr_device_status() == 0


def test_deterministic_and_unsupported_shapes():
    wl, lr, dict_, feat, wconv, bias = _make(CASES[8])
    folded = sr.sr_producer_fold(dev(wconv), dev(bias), dev(dict_), wl.scale, wl.k)
    a = sr.sr_producer_regress(dev(lr), torch.from_numpy(feat).cuda(), folded, wl.scale, wl.k, wl.D, 3)
    b = sr.sr_producer_regress(dev(lr), torch.from_numpy(feat).cuda(), folded, wl.scale, wl.k, wl.D, 3)
    assert torch.equal(a, b)
    w3 = sr_inputs.Workload("t", 1, 3, 8, 32, 3, D=8, k=7)
    f3, wc3, b3 = sr_inputs.make_producer(w3, cin=32, kc=3)
    with pytest.raises(sr.SrError):                          # 7 x 7 atoms at scale 3 are not built
        sr.sr_producer_fold(dev(wc3), dev(b3), dev(sr_inputs.make_dictionary(8, 7)), 3, 7)
    f16c, wc16, b16 = sr_inputs.make_producer(wl, cin=16, kc=3)
    with pytest.raises(sr.SrError):                          # 16 feature channels are not built
        sr.sr_producer_fold(dev(wc16), dev(b16), dev(dict_), wl.scale, wl.k)


def test_a_lost_copy_times_out_and_the_next_call_is_correct():
    wl, lr, dict_, feat, wconv, bias = _make(CASES[0])
    folded = sr.sr_producer_fold(dev(wconv), dev(bias), dev(dict_), wl.scale, wl.k)
    dlr, dfe = dev(lr), torch.from_numpy(feat).cuda()
    good = sr.sr_producer_regress(dlr, dfe, folded, wl.scale, wl.k, wl.D, 3)
    old = sr.sr_set_wait_limit(2_000_000)                     # about a millisecond
    try:
        sr.sr_test_lose_arrival(1)
        sr.sr_producer_regress(dlr, dfe, folded, wl.scale, wl.k, wl.D, 3)
        torch.cuda.synchronize()
        assert sr.sr_device_status() == sr.api.SR_ERR_TIMEOUT
        assert sr.sr_device_status() == 0
    finally:
        sr.sr_set_wait_limit(old)
        sr.sr_test_lose_arrival(0)
    again = sr.sr_producer_regress(dlr, dfe, folded, wl.scale, wl.k, wl.D, 3)
    assert torch.equal(again, good)


@pytest.mark.parametrize("name", ["cfg1", "cfg3", "cfg4"])
def test_full_size_whole_frame(name):
    """The 1080p x4 frame of the benchmark, one frame of the 4K x2 batch and the x3 anchor of the sweep (360 x 640 LR),
    element by element over the whole output,
    in the launch configuration bench.py times (signed, asymmetric dictionary)."""
    from dataclasses import replace
    wl = replace(sr_inputs.CONFIGS[name], n=1)
    lr, dict_, _ = sr_inputs.make_inputs(replace(wl, D=1))      # the coefficient tensor is not needed here
    dict_ = signed_asymmetric_dictionary(sr_inputs.make_dictionary(wl.D, wl.k))
    feat, wconv, bias = sr_inputs.make_producer(wl, cin=32, kc=3)
    folded = sr.sr_producer_fold(dev(wconv), dev(bias), dev(dict_), wl.scale, wl.k)
    got = sr.sr_producer_regress(dev(lr), torch.from_numpy(feat).cuda(), folded, wl.scale, wl.k, wl.D, 3, sr.SR_CLAMP01)
    want = oracle.producer_regress(lr, feat, wconv, bias, dict_, wl.scale, wl.k, flags=oracle.CLAMP01)
    err = np.abs(host(got) - want).max()
    assert err <= TIGHT, err
    assert sr.sr_device_status() == 0
