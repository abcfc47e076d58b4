"""HostPipeline: a stream of frames from host buffers gives, per frame, exactly what the direct device call gives.

Frames differ from step to step and there are more steps than slots, so a slot reused too early (inputs overwritten
before the kernels ran, results overwritten before they were copied out) shows as a wrong frame.
"""
import numpy as np
import pytest
import torch

import paper_2303_08999_b200 as sr
import sr_inputs
from paper_2303_08999_b200.hostpipe import HostPipeline

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("depth", [1, 2, 3])
def test_pipeline_matches_direct_calls(depth):
    wl = sr_inputs.Workload("pipe", 1, 3, 40, 64, 4, 24, 5, "f16", 4)
    steps = 5
    frames = [sr_inputs.make_inputs(wl, seed=70 + i) for i in range(steps)]
    dict_ = torch.from_numpy(frames[0][1]).cuda()
    r, k, s = wl.scale, wl.k, wl.s
    shape_out = (wl.n, wl.c, wl.H, wl.W)

    def work(i, o):
        sr.sr_dict_regress_dense(i["lr"], i["coef"], dict_, r, k, 0, out=o["dense"])
        sr.sr_dict_regress_selected(i["lr"], i["coef"], None, None, dict_, r, k, s, 0, out=o["fused"])

    h_in = [{"lr": torch.from_numpy(f[0]).pin_memory(), "coef": torch.from_numpy(f[2]).pin_memory()} for f in frames]
    h_out = [{p: torch.empty(shape_out, dtype=torch.float32).pin_memory() for p in ("dense", "fused")}
             for _ in range(steps)]
    pipe = HostPipeline({"lr": (tuple(h_in[0]["lr"].shape), torch.float32),
                         "coef": (tuple(h_in[0]["coef"].shape), h_in[0]["coef"].dtype)},
                        {p: (shape_out, torch.float32) for p in ("dense", "fused")}, depth=depth)
    done = [pipe.submit(h_in[i], h_out[i], work) for i in range(steps)]
    pipe.drain()
    torch.cuda.synchronize()
    assert all(e.query() for e in done)
    assert sr.sr_device_status() == 0
    for i in range(steps):
        d_in = {k_: v.cuda() for k_, v in h_in[i].items()}
        d_out = {p: torch.empty(shape_out, dtype=torch.float32, device="cuda") for p in ("dense", "fused")}
        work(d_in, d_out)
        torch.cuda.synchronize()
        for p in d_out:
            assert np.array_equal(h_out[i][p].numpy(), d_out[p].cpu().numpy()), (i, p)
    # consecutive frames really differ, so the comparison above can tell them apart
    assert not np.array_equal(h_out[0]["dense"].numpy(), h_out[1]["dense"].numpy())


def test_pipeline_rejects_bad_depth():
    with pytest.raises(ValueError):
        HostPipeline({}, {}, depth=0)
