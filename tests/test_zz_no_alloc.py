"""sr_selection_gram_static: the Gram statistics of the dictionary selection search for callers that must not allocate.

Some users of the library cannot call the device allocator where they need these statistics (a pipeline that fixes its
buffers at start-up and runs under a memory budget, a plug-in inside an application that owns the allocator). For them
the entry point keeps its per-block partial sums in a device array that belongs to the library (at most 80 atoms)
instead of in scratch memory the caller passes. This file calls it through the C ABI exactly as such a caller would
(raw pointers, no wrapper) and checks it against the ordinary entry point, sr_selection_gram, which gets its scratch
from the caller: same inputs, same outputs within the tolerance of the Gram parity tests (the two differ only in how
many blocks share the work, i.e. in the grouping of the fp64 sums). Two calls in a row on different inputs show that
nothing of the first call survives in the shared array, and the device's free memory does not move across the calls.

The file name sorts last on purpose: a run that stops at its first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import dev, host, signed_asymmetric_dictionary
from paper_2303_08999_b200 import api

pytestmark = pytest.mark.gpu


def _inputs(D, k, r, h, w, seed, n=1, c=3):
    wl = sr_inputs.Workload("t", n, c, h, w, r, D=D, k=k, coef_dtype="f16")
    lr, d, coef = sr_inputs.make_inputs(wl, seed=sr_inputs.BASE_SEED + seed)
    d = signed_asymmetric_dictionary(d, seed=seed)
    target = oracle.dict_regress_dense(lr, coef, d, r, k).astype(np.float32)
    return wl, tuple(dev(a) for a in (lr, coef, d, target))


def _static_call(lib, wl, lr, coef, d, target, samples, flags=0):
    """The call a caller without an allocator makes: every buffer is one it already owns."""
    D = wl.D
    G = torch.full((D, D), float("nan"), dtype=torch.float64, device="cuda")
    b = torch.full((D,), float("nan"), dtype=torch.float64, device="cuda")
    hh = torch.full((1,), float("nan"), dtype=torch.float64, device="cuda")
    dims = api.sr_dims(wl.n, wl.c, wl.h, wl.w, wl.scale, wl.k, D)
    status = lib.sr_selection_gram_static(lr.data_ptr(), coef.data_ptr(), api.SR_F16, d.data_ptr(), target.data_ptr(),
                                          None if samples is None else samples.data_ptr(), 0 if samples is None else samples.numel(),
                                          G.data_ptr(), b.data_ptr(), hh.data_ptr(), ctypes.byref(dims), flags,
                                          torch.cuda.current_stream().cuda_stream)
    return status, G, b, hh


def _close(got, want):
    """Tolerance of the Gram parity tests (tests/test_gpu_selection.py), here between the two entry points."""
    G, b, hh = (host(t) for t in got)
    wG, wb, whh = (host(t) for t in want)
    dg = np.sqrt(np.diag(wG))
    assert np.all(np.abs(G - wG) <= 2e-5 * np.outer(dg, dg) + 1e-30)
    assert np.all(np.abs(b - wb) <= 2e-5 * dg * np.sqrt(whh[0]) + 1e-30)
    assert abs(hh[0] - whh[0]) <= 1e-6 * whh[0]


def test_static_scratch_entry_point_matches_the_ordinary_one_on_two_calls_in_a_row():
    lib = sr.load_library()
    wl_a, in_a = _inputs(72, 5, 4, 12, 16, seed=1)
    wl_b, in_b = _inputs(24, 3, 2, 20, 9, seed=2, n=2)        # fewer atoms, fewer pixels: parts of the array keep call A's sums
    samples_b = dev(np.random.default_rng(3).integers(0, wl_b.npix, size=301, dtype=np.int64))
    want_a = sr.sr_selection_gram(*in_a, None, wl_a.scale, wl_a.k)
    want_b = sr.sr_selection_gram(*in_b, samples_b, wl_b.scale, wl_b.k)
    st, *got = _static_call(lib, wl_a, *in_a, None)           # the first call on the device also looks up the array's address
    assert st == api.SR_OK
    _close(got, want_a)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    st, *got_b = _static_call(lib, wl_b, *in_b, samples_b)
    assert st == api.SR_OK
    st, *got_a2 = _static_call(lib, wl_a, *in_a, None)
    assert st == api.SR_OK
    torch.cuda.synchronize()
    _close(got_b, want_b)
    _close(got_a2, want_a)
    assert all(torch.equal(x, y) for x, y in zip(got, got_a2))           # same inputs, same bits, whatever ran in between
    # the outputs above were allocated by this test before the calls; the calls themselves took no device memory
    assert torch.cuda.mem_get_info()[0] >= free_before - 3 * (72 * 72 + 72 + 1) * 8 - (1 << 21)
    assert sr.sr_device_status() == 0


def test_static_scratch_entry_point_rejects_what_its_array_cannot_hold():
    lib = sr.load_library()
    wl, ins = _inputs(96, 3, 2, 6, 6, seed=4)
    st, G, b, hh = _static_call(lib, wl, *ins, None)
    assert st == api.SR_ERR_TOO_LARGE and "built-in scratch" in sr.status_string(st)
    assert bool(torch.isnan(G).all()) and bool(torch.isnan(hh).all())    # nothing was launched
    wl, ins = _inputs(80, 3, 2, 6, 6, seed=5)                             # the limit itself is fine
    st, *got = _static_call(lib, wl, *ins, None)
    assert st == api.SR_OK
    _close(got, sr.sr_selection_gram(*ins, None, wl.scale, wl.k))
