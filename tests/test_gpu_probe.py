"""Issue-rate probes (the denominators of the ALU- and FMA-bound rooflines): each kind runs, reports a rate in the
range the SM's lane counts allow, and an unknown kind is refused."""
import ctypes

import pytest
import torch

import paper_2303_08999_b200 as sr
from paper_2303_08999_b200 import api

pytestmark = pytest.mark.gpu


def test_probe_rates_are_plausible_and_unknown_kinds_are_refused():
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    top = sms * 128 * 2.2e9                                # 128 fp32 lanes per SM at a clock no B200 reaches
    maxmin, fma, fma2 = (sr.sr_probe_rate(k) for k in (0, 1, 2))
    assert 0.2 * top < maxmin < top                        # max/min issue at half the fp32 lane count
    assert 0.5 * top < fma < top
    assert 0.5 * top < fma2 < top                          # packed form: fewer issue slots, the same lanes
    scratch = torch.zeros(2, dtype=torch.int32, device="cuda")
    v = ctypes.c_double(0.0)
    for bad in (-1, 3):
        assert api.load_library().sr_probe_rate(bad, ctypes.c_void_p(scratch.data_ptr()), ctypes.byref(v), None) == api.SR_ERR_UNSUPPORTED
    assert sr.sr_device_status() == 0
