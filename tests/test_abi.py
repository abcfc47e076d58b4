"""The C-ABI library loads, exports every symbol the public header declares, and validates arguments
on the host before anything is launched (so these calls need no GPU)."""
import ctypes
import os
import re

import pytest

import paper_2303_08999_b200 as sr
from paper_2303_08999_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return sr.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "sr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sr_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert set(api.EXPORTS) <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    seen = {sr.status_string(i) for i in range(8)}
    assert len(seen) == 8 and sr.status_string(0) == "ok" and sr.status_string(99) == "unknown status"


def _dims(**kw):
    base = dict(n=1, c=3, h=4, w=4, scale=2, k=5, D=8)
    base.update(kw)
    return api.sr_dims(*(base[f] for f in ("n", "c", "h", "w", "scale", "k", "D")))


FAKE = 0x1000  # never dereferenced: every call below fails validation before any launch


def test_validation_errors_come_back_before_any_launch(lib):
    dense = lambda d, coef=FAKE, dt=api.SR_F16, flags=0, lr=FAKE: lib.sr_dict_regress_dense(
        lr, coef, dt, FAKE, FAKE, ctypes.byref(d), flags, None)
    assert dense(_dims(), lr=None) == api.SR_ERR_NULL
    assert dense(_dims(k=4)) == api.SR_ERR_UNSUPPORTED
    assert dense(_dims(k=11)) == api.SR_ERR_UNSUPPORTED
    assert dense(_dims(scale=0)) == api.SR_ERR_UNSUPPORTED
    assert dense(_dims(scale=9)) == api.SR_ERR_UNSUPPORTED
    assert dense(_dims(D=257)) == api.SR_ERR_UNSUPPORTED
    assert dense(_dims(D=0)) == api.SR_ERR_SHAPE
    assert dense(_dims(n=0)) == api.SR_ERR_SHAPE
    assert dense(_dims(h=70000, w=70000)) == api.SR_ERR_SHAPE
    assert dense(_dims(), dt=7) == api.SR_ERR_UNSUPPORTED
    assert dense(_dims(), flags=api.SR_IDX_GLOBAL) == api.SR_ERR_UNSUPPORTED
    assert dense(_dims(), coef=FAKE + 1) == api.SR_ERR_ALIGN
    assert dense(_dims(), coef=FAKE + 2, dt=api.SR_F32) == api.SR_ERR_ALIGN
    assert lib.sr_dict_regress_dense(FAKE, FAKE, api.SR_F16, FAKE, FAKE, None, 0, None) == api.SR_ERR_NULL

    assert lib.sr_bicubic_upsample(None, FAKE, ctypes.byref(_dims()), None) == api.SR_ERR_NULL
    assert lib.sr_bicubic_upsample(FAKE, FAKE + 2, ctypes.byref(_dims()), None) == api.SR_ERR_ALIGN
    assert lib.sr_bicubic_upsample(FAKE, FAKE, ctypes.byref(_dims(scale=12)), None) == api.SR_ERR_UNSUPPORTED
    assert lib.sr_bilinear_upsample(None, FAKE, ctypes.byref(_dims()), None) == api.SR_ERR_NULL
    assert lib.sr_bilinear_upsample(FAKE + 1, FAKE, ctypes.byref(_dims()), None) == api.SR_ERR_ALIGN
    assert lib.sr_bilinear_upsample(FAKE, FAKE, ctypes.byref(_dims(scale=0)), None) == api.SR_ERR_UNSUPPORTED
    # the up-sampling variant is a legal flag of the regression calls: validation goes on to the next check
    assert dense(_dims(k=4), flags=api.SR_UPSAMPLE_BILINEAR) == api.SR_ERR_UNSUPPORTED
    assert dense(_dims(), flags=api.SR_UPSAMPLE_BILINEAR | api.SR_CLAMP01, coef=FAKE + 1) == api.SR_ERR_ALIGN
    assert dense(_dims(), flags=128) == api.SR_ERR_UNSUPPORTED                     # an unknown flag
    assert dense(_dims(c=1), flags=api.SR_LUMA_ONLY) == api.SR_ERR_UNSUPPORTED     # luma-only needs R, G, B planes
    assert dense(_dims(c=3), flags=api.SR_LUMA_ONLY, coef=FAKE + 1) == api.SR_ERR_ALIGN   # legal with c = 3: next check
    assert dense(_dims(), flags=api.SR_OUT_F16 | api.SR_OUT_U8) == api.SR_ERR_UNSUPPORTED   # one output type at a time
    # binary16 output: `out` needs 2-byte alignment only (FAKE + 2 passes this check and fails the next one)
    out_at = lambda out, flags: lib.sr_dict_regress_dense(FAKE, FAKE + 1, api.SR_F16, FAKE, out, ctypes.byref(_dims()), flags, None)
    assert lib.sr_dict_regress_dense(FAKE, FAKE, api.SR_F16, FAKE, FAKE + 2, ctypes.byref(_dims()), 0, None) == api.SR_ERR_ALIGN
    assert lib.sr_dict_regress_dense(FAKE, FAKE, api.SR_F16, FAKE, FAKE + 1, ctypes.byref(_dims()), api.SR_OUT_F16, None) == api.SR_ERR_ALIGN
    assert out_at(FAKE + 2, api.SR_OUT_F16) == api.SR_ERR_ALIGN      # from the odd coefficient pointer, not from `out`

    select = lambda d, s, flags=0, idx=FAKE: lib.sr_dict_select(FAKE, api.SR_F16, idx, None, ctypes.byref(d), s, flags, None)
    assert select(_dims(), 0) == api.SR_ERR_SHAPE
    assert select(_dims(), 9) == api.SR_ERR_SHAPE
    assert select(_dims(), 4, flags=1) == api.SR_ERR_UNSUPPORTED
    assert select(_dims(), 4, idx=None) == api.SR_ERR_NULL

    selected = lambda d, s, flags=0, idx=FAKE, gamma=None: lib.sr_dict_regress_selected(
        FAKE, FAKE, api.SR_F16, idx, gamma, FAKE, FAKE, ctypes.byref(d), s, flags, None)
    assert selected(_dims(), 9) == api.SR_ERR_SHAPE
    assert selected(_dims(), 4, flags=api.SR_IDX_GLOBAL, idx=None) == api.SR_ERR_NULL
    assert selected(_dims(), 4, flags=api.SR_COEF_COMPACT, idx=None) == api.SR_ERR_NULL
    assert selected(_dims(), 4, gamma=FAKE) == api.SR_ERR_UNSUPPORTED  # gamma only exists for the global subset
    assert selected(_dims(), 4, flags=128) == api.SR_ERR_UNSUPPORTED
    assert selected(_dims(c=1), 4, flags=api.SR_LUMA_ONLY) == api.SR_ERR_UNSUPPORTED
    assert lib.sr_device_status(None, None) == api.SR_ERR_NULL

    # the producer-fused calls: pointers and shapes are validated before anything touches the device; without a
    # device that can run the kernel the size query answers 0 and the calls refuse the shape
    d = _dims(scale=4)
    assert lib.sr_producer_fold(None, None, FAKE, None, None, 0, FAKE, 16, ctypes.byref(d), 32, 3, None) == api.SR_ERR_NULL
    assert lib.sr_producer_fold(FAKE, None, FAKE, None, FAKE, 0, FAKE, 16, ctypes.byref(d), 32, 3, None) == api.SR_ERR_UNSUPPORTED  # gamma without idx
    assert lib.sr_producer_fold(FAKE, None, FAKE, FAKE, None, 99, FAKE, 16, ctypes.byref(d), 32, 3, None) == api.SR_ERR_SHAPE
    assert lib.sr_producer_regress(FAKE, None, FAKE, 16, FAKE, ctypes.byref(d), 32, 3, 0, None) == api.SR_ERR_NULL
    assert lib.sr_producer_regress(FAKE, FAKE, FAKE, 16, FAKE, ctypes.byref(d), 32, 3, api.SR_LUMA_ONLY, None) == api.SR_ERR_UNSUPPORTED
    assert lib.sr_producer_regress(FAKE, FAKE, FAKE, 16, FAKE, ctypes.byref(_dims(scale=5)), 32, 3, 0, None) == api.SR_ERR_UNSUPPORTED
    assert lib.sr_producer_folded_bytes(ctypes.byref(_dims(scale=5)), 32, 3) == 0
    assert lib.sr_producer_folded_bytes(ctypes.byref(d), 16, 3) == 0


def test_binding_refuses_cpu_tensors():
    import torch
    with pytest.raises(TypeError):
        sr.sr_bicubic_upsample(torch.zeros(1, 1, 2, 2), 2)
    with pytest.raises(TypeError):
        sr.sr_bilinear_upsample(torch.zeros(1, 1, 2, 2), 2)


def test_wait_limit_is_returned_and_the_hook_validates_its_count(lib):
    old = sr.sr_set_wait_limit(12345)
    assert sr.sr_set_wait_limit(0) == 12345      # < 1: nothing changes, the current budget comes back
    assert sr.sr_set_wait_limit(old) == 12345
    assert lib.sr_test_lose_arrival(-1) == api.SR_ERR_SHAPE
    assert lib.sr_test_lose_arrival(0) == api.SR_OK
    assert lib.sr_test_force_kernel(5) == api.SR_ERR_SHAPE and lib.sr_test_force_kernel(-2) == api.SR_ERR_SHAPE
    assert lib.sr_test_force_kernel(-1) == api.SR_OK
