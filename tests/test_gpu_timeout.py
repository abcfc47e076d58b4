"""The failure path of the bounded device-side waits, exercised without faulting or hanging anything.

A host-side hook makes one producer thread of the first thread block leave out one barrier arrival; with a wait budget
of about a millisecond the consumer's wait runs out, the block raises its abort flag, every other wait of the block
returns, the block drains its copies and tensor-core operations, frees its tensor memory and exits. The host then
reads SR_ERR_TIMEOUT from the status word, the word clears, and the next ordinary call is bit-identical to one made
before the failure (nothing was left behind: tensor memory, barriers, copies in flight).
"""
import numpy as np
import pytest
import torch

import paper_2303_08999_b200 as sr
import sr_inputs
from gpu_util import dev

pytestmark = pytest.mark.gpu

SHORT_BUDGET = 2_000_000   # SM cycles: about a millisecond


def _on_kernel(kernel, fn):
    sr.sr_test_force_kernel(kernel)
    try:
        return fn()
    finally:
        sr.sr_test_force_kernel(-1)


def _calls():
    wl = sr_inputs.Workload("t", 1, 3, 24, 64, 2, D=72, k=5, coef_dtype="f16")
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    dlr, dco, ddi = dev(lr), dev(coef), dev(dict_)
    idx, sel = sr.sr_dict_select(dco, 8, want_sel=True)
    S = dev(np.arange(0, 72, 6, dtype=np.uint8))          # twelve atoms: more than the FMA-pipe subset kernel (no waits) takes
    return {
        "dense": lambda: sr.sr_dict_regress_dense(dlr, dco, ddi, 2, 5),
        "fused_select": lambda: sr.sr_dict_regress_selected(dlr, dco, None, None, ddi, 2, 5, 8),
        "index_planes": lambda: sr.sr_dict_regress_selected(dlr, dco, idx, None, ddi, 2, 5, 8),
        # pinned to the first tensor-core layout: the host rules give this shape to the gather kernel, which has no waits
        "compact": lambda: _on_kernel(1, lambda: sr.sr_dict_regress_selected(dlr, sel, idx, None, ddi, 2, 5, 8, sr.SR_COEF_COMPACT)),
        "global_subset": lambda: sr.sr_dict_regress_selected(dlr, dco, S, None, ddi, 2, 5, 12, sr.SR_IDX_GLOBAL),
        "dense_few_atoms": lambda: sr.sr_dict_regress_dense(dlr, dco[:, :16].contiguous(), ddi[:16].contiguous(), 2, 5),
    }


@pytest.mark.parametrize("mode", ["dense", "fused_select", "index_planes", "compact", "global_subset", "dense_few_atoms"])
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_clean(mode):
    call = _calls()[mode]
    before = call().clone()
    assert sr.sr_device_status() == sr.api.SR_OK
    old = sr.sr_set_wait_limit(SHORT_BUDGET)
    try:
        sr.sr_test_lose_arrival(1)
        call()                                              # returns SR_OK: the failure happens on the device
        assert sr.sr_device_status() == sr.api.SR_ERR_TIMEOUT
        assert sr.sr_device_status() == sr.api.SR_OK        # reading cleared the word
    finally:
        sr.sr_test_lose_arrival(0)
        assert sr.sr_set_wait_limit(old) == SHORT_BUDGET
    for _ in range(2):
        assert torch.equal(call(), before)
    assert sr.sr_device_status() == sr.api.SR_OK
