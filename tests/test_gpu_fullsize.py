"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot run whole 1080p / 4K frames in test time, so outputs are compared at sampled HR
pixels (corners, borders and a seeded random set) that the oracle evaluates one by one, plus
properties that hold at any size (index planes are distinct atoms in non-increasing magnitude order).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, dev, host

pytestmark = pytest.mark.gpu


def _samples(wl, count, seed=11):
    rng = np.random.default_rng(seed)
    H, W = wl.H, wl.W
    s = rng.integers(0, wl.npix, size=count, dtype=np.int64)
    border = []
    for f in range(wl.n):
        base = f * H * W
        for y in (0, 1, 2, H // 2, H - 3, H - 2, H - 1):
            for x in (0, 1, 2, 127, 128, W // 2, W - 3, W - 2, W - 1):
                border.append(base + y * W + x)
    return np.unique(np.concatenate([s, np.array(border, dtype=np.int64)]))


def _gather(t: torch.Tensor, samples, wl):
    """t is [n][planes][H][W] on the device -> [nsamples][planes] on the host."""
    n, planes = t.shape[0], t.shape[1]
    flat = t.reshape(n, planes, -1)
    sm = torch.from_numpy(samples).cuda()
    f, pix = sm // (wl.H * wl.W), sm % (wl.H * wl.W)
    return flat[f, :, pix].cpu().numpy()


def _check_workload(wl, nsamples):
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    samples = _samples(wl, nsamples)
    dlr, ddi = dev(lr), dev(dict_)
    dco = torch.from_numpy(coef).cuda()
    r, k, s = wl.scale, wl.k, wl.s
    flags = sr.SR_CLAMP01

    up = sr.sr_bicubic_upsample(dlr, r)                      # stage 1 alone: the whole frame against the oracle
    err = np.abs(host(up).astype(np.float64) - oracle.bicubic_upsample(lr, r)).max()
    assert err <= 2e-6, f"bicubic {err}"
    del up

    out = sr.sr_dict_regress_dense(dlr, dco, ddi, r, k, flags)
    want = oracle.regress_at("dense", lr, coef, None, None, dict_, samples, r, k, flags=oracle.CLAMP01)
    err = np.abs(_gather(out, samples, wl) - want).max()
    assert err <= TOL_F16, f"dense {err}"
    assert bool(torch.isfinite(out).all())
    del out

    idx, sel = sr.sr_dict_select(dco, s, want_sel=True)
    want_idx = oracle.dict_select_at(coef, samples, s)
    np.testing.assert_array_equal(_gather(idx, samples, wl), want_idx)
    # properties over the whole frame: magnitudes non-increasing in rank, atoms distinct, values match the tensor
    mag = sel.abs()
    assert bool((mag[:, :-1] >= mag[:, 1:]).all())
    srt = idx.sort(dim=1).values
    assert bool((srt[:, 1:] != srt[:, :-1]).all())
    assert bool((torch.gather(dco, 1, idx.long()) == sel).all())

    want = oracle.regress_at("selected", lr, coef, None, None, dict_, samples, r, k, s=s, flags=oracle.CLAMP01)
    out = sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s, flags)
    err = np.abs(_gather(out, samples, wl) - want).max()
    assert err <= TOL_F16, f"fused selected {err}"
    out = sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, s, flags | sr.SR_COEF_COMPACT)
    err = np.abs(_gather(out, samples, wl) - want).max()
    assert err <= TOL_F16, f"compact selected {err}"
    out = sr.sr_dict_regress_selected(dlr, dco, idx, None, ddi, r, k, s, flags)
    err = np.abs(_gather(out, samples, wl) - want).max()
    assert err <= TOL_F16, f"index-listed selected {err}"
    del out, idx, sel

    S = np.arange(0, wl.D, wl.D // s, dtype=np.uint8)[:s]
    gamma = np.linspace(0.75, 1.25, s).astype(np.float32)
    want = oracle.regress_at("selected", lr, coef, S, gamma, dict_, samples, r, k, s=s,
                             flags=oracle.CLAMP01 | oracle.IDX_GLOBAL)
    out = sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, s, flags | sr.SR_IDX_GLOBAL)
    err = np.abs(_gather(out, samples, wl) - want).max()
    assert err <= TOL_F16, f"global subset {err}"
    assert sr.sr_device_status() == 0


def test_cfg1_cfg2_1080p_x4():
    _check_workload(sr_inputs.CONFIGS["cfg1"], 20000)


def test_cfg3_batch_of_four_4k_x2():
    _check_workload(sr_inputs.CONFIGS["cfg3"], 20000)


@pytest.mark.parametrize("wl", [w for w in sr_inputs.cfg4_points()
                                if (w.scale, w.D, w.k) in {(2, 16, 3), (3, 32, 7), (4, 128, 5), (3, 72, 5), (2, 128, 7), (4, 16, 7)}],
                         ids=lambda w: w.name)
def test_cfg4_sweep_points(wl):
    for s in (4, 8, 16):
        if s > wl.D:
            continue
        from dataclasses import replace
        _check_workload(replace(wl, s=s), 4000)
