"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The 1080p x4 frame (cfg1 / cfg2) and the batch of four 4K frames (cfg3) are compared with the oracle over the WHOLE
output, element by element, for every path of a benchmark step (the oracle needs about a second per path and frame
on the host cores). The 36 points of the shape sweep (cfg4) are compared on more than 20 000 sampled pixels each,
which include every tile-seam row and column, evaluated one by one by the oracle. Two dictionaries are used: the
generator's Gaussian / difference-of-Gaussians atoms, and the same atoms made asymmetric and signed (a tap flip or a
lost sign shows only with those).
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, dev, host, signed_asymmetric_dictionary, signed_gamma

pytestmark = pytest.mark.gpu


def _err(got: torch.Tensor, want: np.ndarray) -> float:
    return float(np.abs(host(got).astype(np.float64) - want).max())


def _subset(wl):
    S = np.arange(0, wl.D, max(1, wl.D // wl.s), dtype=np.uint8)[: wl.s]
    return S, signed_gamma(wl.s)


def _whole_frames(wl, signed: bool, paths):
    """Every listed path over whole frames, frame by frame (bounds the oracle's fp64 outputs to one frame)."""
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    if signed:
        dict_ = signed_asymmetric_dictionary(dict_)
    r, k, s = wl.scale, wl.k, wl.s
    fl, ofl = sr.SR_CLAMP01, oracle.CLAMP01
    ddi = dev(dict_)
    S, gamma = _subset(wl)
    for f in range(wl.n):
        lr1, co1 = lr[f:f + 1], coef[f:f + 1]
        dlr, dco = dev(lr1), torch.from_numpy(co1).cuda()
        if "bicubic" in paths:
            assert _err(sr.sr_bicubic_upsample(dlr, r), oracle.bicubic_upsample(lr1, r)) <= 2e-6
        if "dense" in paths:
            e = _err(sr.sr_dict_regress_dense(dlr, dco, ddi, r, k, fl), oracle.dict_regress_dense(lr1, co1, dict_, r, k, flags=ofl))
            assert e <= TOL_F16, f"dense, frame {f}: {e}"
        idx = sel = None
        if "select" in paths:
            idx, sel = sr.sr_dict_select(dco, s, want_sel=True)
            want_idx, want_sel = oracle.dict_select(co1, s, want_sel=True)
            np.testing.assert_array_equal(host(idx), want_idx)
            np.testing.assert_array_equal(host(sel).astype(np.float64), want_sel)
        if {"fused", "compact", "idx"} & set(paths):
            want = oracle.dict_regress_selected(lr1, co1, None, None, dict_, r, k, s, flags=ofl)
            if "fused" in paths:
                e = _err(sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s, fl), want)
                assert e <= TOL_F16, f"fused selection, frame {f}: {e}"
            if "compact" in paths:
                e = _err(sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, s, fl | sr.SR_COEF_COMPACT), want)
                assert e <= TOL_F16, f"compact, frame {f}: {e}"
            if "idx" in paths:
                e = _err(sr.sr_dict_regress_selected(dlr, dco, idx, None, ddi, r, k, s, fl), want)
                assert e <= TOL_F16, f"index-listed, frame {f}: {e}"
            del want
        if "global" in paths:
            want = oracle.dict_regress_selected(lr1, co1, S, gamma, dict_, r, k, s, flags=ofl | oracle.IDX_GLOBAL)
            e = _err(sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, s, fl | sr.SR_IDX_GLOBAL), want)
            assert e <= TOL_F16, f"global subset, frame {f}: {e}"
        del dlr, dco, idx, sel
    assert sr.sr_device_status() == 0


ALL_PATHS = ("bicubic", "dense", "select", "fused", "compact", "idx", "global")


@pytest.mark.parametrize("signed", [False, True], ids=["generator_atoms", "signed_asymmetric_atoms"])
def test_cfg1_cfg2_1080p_x4_whole_frame_every_path(signed):
    _whole_frames(sr_inputs.CONFIGS["cfg1"], signed, ALL_PATHS)


def test_cfg3_batch_of_four_4k_x2_whole_batch():
    """One launch per call over the whole batch is what the benchmark times; here the four frames also go through one
    by one so that the oracle's outputs stay bounded, and the batched launch is checked to give the same bits."""
    wl = sr_inputs.CONFIGS["cfg3"]
    _whole_frames(wl, True, ("dense", "fused", "select", "global"))
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    dict_ = signed_asymmetric_dictionary(dict_)
    r, k, s = wl.scale, wl.k, wl.s
    dlr, ddi = dev(lr), dev(dict_)
    dco = torch.from_numpy(coef).cuda()
    for call in (lambda a, b: sr.sr_dict_regress_dense(a, b, ddi, r, k, sr.SR_CLAMP01),
                 lambda a, b: sr.sr_dict_regress_selected(a, b, None, None, ddi, r, k, s, sr.SR_CLAMP01)):
        batched = call(dlr, dco)
        for f in range(wl.n):
            assert torch.equal(batched[f], call(dlr[f:f + 1].contiguous(), dco[f:f + 1].contiguous())[0])
        del batched
    assert sr.sr_device_status() == 0


def _samples(wl, count, seed=11):
    """Flat [n][H][W] indices: a seeded random set, the frame's corners and borders, and points on both sides of every
    tile seam (tiles are 128 pixels wide and 8 or 16 rows high)."""
    rng = np.random.default_rng(seed)
    H, W = wl.H, wl.W
    pts = [rng.integers(0, wl.npix, size=count, dtype=np.int64)]
    for f in range(wl.n):
        base = f * H * W
        ys = np.array([0, 1, 2, H // 2, H - 3, H - 2, H - 1])
        xs = np.array([0, 1, 2, 127, 128, W // 2, W - 3, W - 2, W - 1])
        pts.append((base + ys[:, None] * W + xs[None, :]).ravel())
        seam_y = np.unique(np.clip(np.concatenate([np.arange(0, H, 8) - 1, np.arange(0, H, 8)]), 0, H - 1))
        xr = rng.integers(0, W, size=(seam_y.size, 6))
        pts.append((base + seam_y[:, None] * W + xr).ravel())
        seam_x = np.unique(np.clip(np.concatenate([np.arange(0, W, 64) - 1, np.arange(0, W, 64)]), 0, W - 1))
        yr = rng.integers(0, H, size=(seam_x.size, 6))
        pts.append((base + yr * W + seam_x[:, None]).ravel())
    return np.unique(np.concatenate(pts).astype(np.int64))


def _gather(t: torch.Tensor, samples, wl):
    """t is [n][planes][H][W] on the device -> [nsamples][planes] on the host."""
    n, planes = t.shape[0], t.shape[1]
    flat = t.reshape(n, planes, -1)
    sm = torch.from_numpy(samples).cuda()
    f, pix = sm // (wl.H * wl.W), sm % (wl.H * wl.W)
    return flat[f, :, pix].cpu().numpy()


@pytest.mark.parametrize("wl", list(sr_inputs.cfg4_points()), ids=lambda w: w.name)
def test_cfg4_every_sweep_point(wl):
    """Dense and s in {4, 8, 16} (s <= D) at every point of the sweep, on sampled pixels."""
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    dict_ = signed_asymmetric_dictionary(dict_)
    samples = _samples(wl, 20000)
    assert samples.size >= 20000
    dlr, ddi = dev(lr), dev(dict_)
    dco = torch.from_numpy(coef).cuda()
    r, k = wl.scale, wl.k
    fl, ofl = sr.SR_CLAMP01, oracle.CLAMP01
    out = sr.sr_dict_regress_dense(dlr, dco, ddi, r, k, fl)
    want = oracle.regress_at("dense", lr, coef, None, None, dict_, samples, r, k, flags=ofl)
    e = np.abs(_gather(out, samples, wl) - want).max()
    assert e <= TOL_F16, f"dense {e}"
    assert bool(torch.isfinite(out).all())
    for s in (4, 8, 16):
        if s > wl.D:
            continue
        idx, sel = sr.sr_dict_select(dco, s, want_sel=True)
        np.testing.assert_array_equal(_gather(idx, samples, wl), oracle.dict_select_at(coef, samples, s))
        # properties over the whole frame: magnitudes non-increasing in rank, atoms distinct, values match the tensor
        mag = sel.abs()
        assert bool((mag[:, :-1] >= mag[:, 1:]).all())
        srt = idx.sort(dim=1).values
        assert bool((srt[:, 1:] != srt[:, :-1]).all())
        assert bool((torch.gather(dco, 1, idx.long()) == sel).all())
        want = oracle.regress_at("selected", lr, coef, None, None, dict_, samples, r, k, s=s, flags=ofl)
        out = sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, r, k, s, fl)
        e = np.abs(_gather(out, samples, wl) - want).max()
        assert e <= TOL_F16, f"fused selection s={s}: {e}"
        out = sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, r, k, s, fl | sr.SR_COEF_COMPACT)
        e = np.abs(_gather(out, samples, wl) - want).max()
        assert e <= TOL_F16, f"compact s={s}: {e}"
        S, gamma = _subset(replace(wl, s=s))
        want = oracle.regress_at("selected", lr, coef, S, gamma, dict_, samples, r, k, s=s, flags=ofl | oracle.IDX_GLOBAL)
        out = sr.sr_dict_regress_selected(dlr, dco, dev(S), dev(gamma), ddi, r, k, s, fl | sr.SR_IDX_GLOBAL)
        e = np.abs(_gather(out, samples, wl) - want).max()
        assert e <= TOL_F16, f"global subset s={s}: {e}"
        assert bool(torch.isfinite(out).all())
    assert sr.sr_device_status() == 0
