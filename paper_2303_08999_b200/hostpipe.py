"""Host-buffer pipeline around the library calls: streams, events and staging buffers only.

A caller whose frames live in host memory pays three things per step: the copy of the inputs to the device, the
kernels, and the copy of the results back.  On the 1080p x4 workload the copies are ten times the kernel time, and the
two directions of the host link are independent, so the throughput of a stream of frames is set by the slower
direction as long as step i+1's inputs travel while step i's results do.  `HostPipeline` does exactly that with
`depth` device-side slots and three streams (copy-in, compute, copy-out) ordered by events; it holds none of the
method's arithmetic, which stays in the kernels the caller's `work` function launches.
"""
from __future__ import annotations

from typing import Callable, Dict, Tuple

import torch


class HostPipeline:
    """`depth` slots of device inputs and outputs, filled and drained on their own streams.

    in_specs / out_specs: name -> (shape, dtype) of the device-side staging tensors of one step.
    """

    def __init__(self, in_specs: Dict[str, Tuple[tuple, torch.dtype]], out_specs: Dict[str, Tuple[tuple, torch.dtype]],
                 depth: int = 2, device=None):
        if not torch.cuda.is_available():
            raise RuntimeError("HostPipeline needs a CUDA device")
        if depth < 1:
            raise ValueError("depth must be at least 1")
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.depth = depth
        self.s_in, self.s_run, self.s_out = (torch.cuda.Stream(self.device) for _ in range(3))
        self.slots = []
        for _ in range(depth):
            self.slots.append({
                "in": {k: torch.empty(sh, dtype=dt, device=self.device) for k, (sh, dt) in in_specs.items()},
                "out": {k: torch.empty(sh, dtype=dt, device=self.device) for k, (sh, dt) in out_specs.items()},
                "in_ready": None, "ran": None, "drained": None,
            })
        self.step = 0

    def submit(self, host_in: Dict[str, torch.Tensor], host_out: Dict[str, torch.Tensor],
               work: Callable[[Dict[str, torch.Tensor], Dict[str, torch.Tensor]], None]) -> torch.cuda.Event:
        """Queues one step and returns the event after which `host_out` holds its results.

        host_in / host_out are pinned host tensors (a pageable one makes its copy synchronous); host_in must stay
        unchanged until the step's inputs have been copied, host_out is written by the copy-out stream.  `work(dev_in,
        dev_out)` launches the step's kernels on the current stream (the compute stream while it runs).
        """
        slot = self.slots[self.step % self.depth]
        self.step += 1
        caller = torch.cuda.current_stream(self.device)
        with torch.cuda.stream(self.s_in):
            self.s_in.wait_stream(caller)                 # whatever produced host_in's contents on the caller's stream
            if slot["ran"] is not None:
                self.s_in.wait_event(slot["ran"])         # the slot's previous step has consumed its inputs
            for k, t in slot["in"].items():
                t.copy_(host_in[k], non_blocking=True)
            slot["in_ready"] = self.s_in.record_event()
        with torch.cuda.stream(self.s_run):
            self.s_run.wait_event(slot["in_ready"])
            if slot["drained"] is not None:
                self.s_run.wait_event(slot["drained"])    # the slot's previous results have left the device
            work(slot["in"], slot["out"])
            slot["ran"] = self.s_run.record_event()
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(slot["ran"])
            for k, t in slot["out"].items():
                host_out[k].copy_(t, non_blocking=True)
            slot["drained"] = self.s_out.record_event()
        return slot["drained"]

    def drain(self) -> None:
        """Makes the caller's current stream wait for everything queued so far."""
        cur = torch.cuda.current_stream(self.device)
        for s in (self.s_in, self.s_run, self.s_out):
            cur.wait_stream(s)
