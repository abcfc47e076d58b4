"""Tile-shape search (Section III-B restated: legal launch shapes from resource constraints, the fastest kept by
measured latency): the search times more than one shape, never records something slower than the host rules' choice,
and whatever it records computes the same regression (within the path's tolerance against the oracle)."""
import numpy as np
import pytest

import oracle
import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import TOL_F16, dev, host, signed_asymmetric_dictionary, signed_gamma

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _forget_recorded_shapes():
    sr.sr_tune_reset()
    yield
    sr.sr_tune_reset()


@pytest.mark.parametrize("D,k,r", [(16, 5, 2), (72, 5, 4), (32, 7, 2)])
def test_dense_search_keeps_the_result_and_never_loses_to_the_host_rules(D, k, r):
    wl = sr_inputs.Workload("t", 1, 3, 80, 96, r, D=D, k=k, coef_dtype="f16")
    lr, d, coef = sr_inputs.make_inputs(wl)
    d = signed_asymmetric_dictionary(d)
    dlr, dco, ddi = dev(lr), dev(coef), dev(d)
    before = host(sr.sr_dict_regress_dense(dlr, dco, ddi, r, k))
    res = sr.sr_tune_dense(dlr, dco, ddi, r, k, reps=3)
    assert res["candidates"] > 1
    assert res["best_us"] <= res["default_us"] * 1.0001
    after = host(sr.sr_dict_regress_dense(dlr, dco, ddi, r, k))
    want = oracle.dict_regress_dense(lr, coef, d, r, k)
    assert np.abs(after - want).max() <= TOL_F16 and np.abs(before - want).max() <= TOL_F16
    sr.sr_tune_reset()
    np.testing.assert_array_equal(host(sr.sr_dict_regress_dense(dlr, dco, ddi, r, k)), before)     # back to the host rules
    assert sr.sr_device_status() == 0


@pytest.mark.parametrize("s", [8, 12])
def test_global_subset_search(s):
    wl = sr_inputs.Workload("t", 1, 3, 48, 64, 4, D=72, k=5, coef_dtype="f16")
    lr, d, coef = sr_inputs.make_inputs(wl)
    d = signed_asymmetric_dictionary(d)
    S = np.arange(0, 72, 72 // s, dtype=np.uint8)[:s]
    gamma = signed_gamma(s)
    args = (dev(lr), dev(coef), dev(S), dev(gamma), dev(d), 4, 5, s, sr.SR_IDX_GLOBAL)
    res = sr.sr_tune_selected(*args, reps=3)
    assert res["candidates"] > 1 and res["best_us"] <= res["default_us"] * 1.0001
    assert res["kernel"] in ("subset (FMA pipe)", "second tensor-core layout", "first tensor-core layout")
    want = oracle.dict_regress_selected(lr, coef, S, gamma, d, 4, 5, s, flags=oracle.IDX_GLOBAL)
    assert np.abs(host(sr.sr_dict_regress_selected(*args)) - want).max() <= TOL_F16
    # a shape that has only one way to run is still accepted
    one = sr.sr_tune_selected(dev(lr), dev(coef.astype(np.float32)), None, None, dev(d), 4, 5, s, 0, reps=1)
    assert one["candidates"] == 1 and one["kernel"] == "general"
    assert sr.sr_device_status() == 0
