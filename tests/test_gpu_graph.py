"""The calls allocate nothing and never synchronise the host, so a step of them can be recorded into a CUDA graph
once and replayed on new frame contents (video streaming: one graph launch per frame instead of six calls).

The test records all six calls of a step after one ordinary warm-up step (the first launch of a kernel on a device
sets its shared-memory attribute; that belongs before the recording), replays the graph on two other frames copied
into the recorded input buffers, and compares every output bit for bit with ordinary calls on the same frames.
"""
import numpy as np
import pytest
import torch

import paper_2303_08999_b200 as sr
import sr_inputs

pytestmark = pytest.mark.gpu


def test_step_replays_from_a_cuda_graph():
    wl = sr_inputs.Workload("graph", 1, 3, 32, 48, 4, 72, 5, "f16", 8)
    frames = [sr_inputs.make_inputs(wl, seed=300 + i) for i in range(3)]
    r, k, s = wl.scale, wl.k, wl.s
    dict_ = torch.from_numpy(frames[0][1]).cuda()
    S = torch.arange(0, 72, 9, dtype=torch.uint8, device="cuda")
    gamma = torch.linspace(0.75, 1.25, 8, device="cuda")
    shape = (wl.n, wl.c, wl.H, wl.W)

    def buffers():
        o = {p: torch.empty(shape, dtype=torch.float32, device="cuda") for p in ("up", "dense", "compact", "fused", "global")}
        o["idx"] = torch.empty((wl.n, s, wl.H, wl.W), dtype=torch.uint8, device="cuda")
        o["sel"] = torch.empty((wl.n, s, wl.H, wl.W), dtype=torch.float16, device="cuda")
        return o

    def step(lr, coef, o):
        sr.sr_bicubic_upsample(lr, r, out=o["up"])
        sr.sr_dict_regress_dense(lr, coef, dict_, r, k, sr.SR_CLAMP01, out=o["dense"])
        sr.sr_dict_select(coef, s, idx=o["idx"], sel=o["sel"])
        sr.sr_dict_regress_selected(lr, o["sel"], o["idx"], None, dict_, r, k, s, sr.SR_CLAMP01 | sr.SR_COEF_COMPACT, out=o["compact"])
        sr.sr_dict_regress_selected(lr, coef, None, None, dict_, r, k, s, sr.SR_CLAMP01, out=o["fused"])
        sr.sr_dict_regress_selected(lr, coef, S, gamma, dict_, r, k, s, sr.SR_CLAMP01 | sr.SR_IDX_GLOBAL, out=o["global"])

    g_lr = torch.from_numpy(frames[0][0]).cuda()
    g_coef = torch.from_numpy(frames[0][2]).cuda()
    g_out = buffers()
    step(g_lr, g_coef, g_out)                  # warm-up outside the recording
    torch.cuda.synchronize()
    launches0 = sr.sr_launch_count()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step(g_lr, g_coef, g_out)
    assert sr.sr_launch_count() - launches0 == 6   # six kernels recorded, nothing else launched by the library
    for i in (1, 2):
        lr, coef = torch.from_numpy(frames[i][0]).cuda(), torch.from_numpy(frames[i][2]).cuda()
        g_lr.copy_(lr)
        g_coef.copy_(coef)
        graph.replay()
        want = buffers()
        step(lr, coef, want)
        torch.cuda.synchronize()
        for name in want:
            assert torch.equal(g_out[name], want[name]), (i, name)
    assert sr.sr_device_status() == 0
    assert not torch.equal(g_out["dense"], torch.zeros_like(g_out["dense"]))
