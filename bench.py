#!/usr/bin/env python
"""Benchmark of the dictionary-regression hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg1]

One step = one pass of the whole hot path over one frame batch of the workload (default: the
1080p-output x4 frame, LR 3x270x480, D=72 atoms of 5x5, binary16 coefficients), i.e. six library
calls on one stream:
    bicubic    sr_bicubic_upsample                           (stage 1 alone)
    dense      sr_dict_regress_dense                         (up-sample + assemble + filter, fused)
    select     sr_dict_select (indices + selected values)
    compact    sr_dict_regress_selected from those index / value planes
    fused      sr_dict_regress_selected with idx = NULL      (select + regress in one call)
    global     sr_dict_regress_selected with one atom subset + re-weights (the paper's structured form)
`value` is HR megapixels per second of whole steps (all N GPUs together; every rank owns its own
frames and nothing is exchanged: weak scaling, no collective on the data path). Per-path times, the
roofline of the dominant kernel and the CPU oracle timed on a bounded sample are reported beside it.
Order of a run: W warm-up steps; K steps with a CUDA event between every call (per-path times, names the
slowest path); then the timed region, exactly K steps with events only around the slowest path's call
(an event record costs about 3 us of stream time; the roofline kernel's duration comes from these).

`--impl reference` times the CPU oracle (test infrastructure, fp64, as it stands) on the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

PATHS = ("bicubic", "dense", "select", "compact", "fused", "global")
METRIC = "HR megapixels/s"


def algorithmic_bytes_per_pixel(wl, path: str) -> float:
    """Bytes that must cross HBM per HR pixel: coefficients read once, output written once, LR read once."""
    cb = 2 if wl.coef_dtype == "f16" else 4
    io = 4 * wl.c + 4 * wl.c / (wl.scale ** 2)
    s, D = wl.s, wl.D
    return {
        "bicubic": io,                             # LR read, up-sampled frame written
        "dense": D * cb + io,
        "select": D * cb + s + s * cb,            # read all planes, write uint8 indices and selected values
        "compact": s * (cb + 1) + io,             # read index + value planes
        "fused": D * cb + io,
        "global": s * cb + io,                    # only the subset's planes are read
    }[path]


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank owns its own frames: the generator seed is offset by the rank (weak scaling, no data exchange)."""
    return base_seed + rank


def max_over_ranks(value_ms: float, dist=None, device=None) -> float:
    """Device time of the slowest rank (the only collective on the timing path); identity without a process group."""
    if dist is None or not dist.is_initialized():
        return float(value_ms)
    import torch
    t = torch.tensor([value_ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, pixels_per_rank_step: int, steps: int, max_ms: float) -> float:
    """HR megapixels per second of the whole job: all ranks' pixels over the slowest rank's time."""
    return world * pixels_per_rank_step * steps / (max_ms * 1e-3) / 1e6


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# DRAM bytes per HR pixel seen by ncu (dram__bytes_read.sum + dram__bytes_write.sum) for each path's
# kernel on the default workload; figures and commands are in profiles/. None = not captured yet.
NCU_TRAFFIC_BYTES_PER_PIXEL = {"bicubic": None, "dense": 154.2, "select": 161.7, "compact": 25.7, "fused": 154.3, "global": 17.0}


# Half-rate ALU-pipe lane operations per HR pixel of the two selection kernels (sorting-network max/min plus the
# logic and address operations that share their pipe, counted from the networks in csrc/sr_select.cu and the select
# role of csrc/sr_umma_impl.inc) and the B200 rate of that
# pipe: 148 SMs x 64 lanes/clk x 1.965 GHz. The fused kernel works on packed binary16 pairs (two pixels per lane
# operation): 315 max/min + 36 logic + 40 address operations per pixel, below its HBM time, so it is HBM-bound.
ALU_OPS_PER_PIXEL = {"select": 630.0, "fused": 391.0}
ALU_PEAK_GOPS = 148 * 64 * 1.965


def path_roofline(wl, path: str, ms: float, hbm_peak: float, peak_kind: str, traffic_bytes_per_pixel):
    """Roofline entry of one path: the slower of its bytes at HBM bandwidth and its selection ops at the ALU rate."""
    by = algorithmic_bytes_per_pixel(wl, path) * wl.npix
    t_hbm = by / (hbm_peak * 1e9)
    ops = ALU_OPS_PER_PIXEL.get(path, 0.0) * wl.npix if (wl.D == 72 and wl.s == 8) else 0.0
    t_alu = ops / (ALU_PEAK_GOPS * 1e9)
    traffic = None if traffic_bytes_per_pixel is None else traffic_bytes_per_pixel * wl.npix
    if t_alu > t_hbm:
        ach = ops / (ms * 1e-3) / 1e9
        return {"kernel": path, "bound": "alu", "achieved": ach, "peak": ALU_PEAK_GOPS, "unit": "Gop/s (max/min lanes)",
                "frac": ach / ALU_PEAK_GOPS, "peak_kind": "derived: 148 SMs x 64 lanes/clk x 1.965 GHz", "traffic": traffic,
                "hbm_frac": by / (ms * 1e-3) / 1e9 / hbm_peak}
    ach = by / (ms * 1e-3) / 1e9
    return {"kernel": path, "bound": "hbm", "achieved": ach, "peak": hbm_peak, "unit": "GB/s", "frac": ach / hbm_peak,
            "peak_kind": f"of {peak_kind}", "traffic": traffic}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs.

    The sampler starts before the warm-up; `stop(t0, t1)` keeps the samples whose timestamps fall inside the timed
    region [t0, t1] (host wall-clock seconds) and falls back to the busiest half when the region was shorter than
    the sampling period.
    """
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_uuid: str | None):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        cmd = ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20"]
        if gpu_uuid:
            cmd += ["-i", gpu_uuid]
        try:
            self.proc = subprocess.Popen(cmd, stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def wait_first_sample(self, timeout_s: float = 5.0):
        t0 = time.time()
        while self.proc is not None and time.time() - t0 < timeout_s:
            if os.path.getsize(self.tmp.name) > 0:
                return
            time.sleep(0.02)

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        import datetime
        rows = []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.tmp.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]), float(parts[3]),
                             [n for n, v in zip(names, parts[4:8]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        self.tmp.close()
        os.unlink(self.tmp.name)
        inside = [r for r in rows if t0 <= r[0] <= t1]
        how = "samples inside the timed region"
        if not inside and rows:
            how = "timed region shorter than the sampling period: busiest half of all samples"
            inside = sorted(rows, key=lambda r: r[1])[len(rows) // 2:]
        reasons = sorted({n for r in inside for n in r[4]})
        return {"sm_mhz": statistics.median([r[1] for r in inside]) if inside else None,
                "sm_max_mhz": max([r[2] for r in rows]) if rows else None,
                "power_w_max": max([r[3] for r in inside]) if inside else None,
                "samples": len(inside), "reasons": reasons, "how": how}


def oracle_step(oracle, wl, lr, dict_, coef, S, gamma, rows: int | None, threads: int = 0):
    """The step's six paths on the CPU oracle, on the top `rows` LR rows of every frame (None = all)."""
    if rows is not None and rows < wl.h:
        lr = lr[:, :, :rows].copy()
        coef = coef[:, :, : rows * wl.scale].copy()
    r, k, s = wl.scale, wl.k, wl.s
    oracle.bicubic_upsample(lr, r, threads=threads)
    oracle.dict_regress_dense(lr, coef, dict_, r, k, flags=oracle.CLAMP01, threads=threads)
    idx, sel = oracle.dict_select(coef, s, want_sel=True, threads=threads)
    sel = sel.astype(coef.dtype)
    oracle.dict_regress_selected(lr, sel, idx, None, dict_, r, k, s, flags=oracle.CLAMP01 | oracle.COEF_COMPACT, threads=threads)
    oracle.dict_regress_selected(lr, coef, None, None, dict_, r, k, s, flags=oracle.CLAMP01, threads=threads)
    oracle.dict_regress_selected(lr, coef, S, gamma, dict_, r, k, s, flags=oracle.CLAMP01 | oracle.IDX_GLOBAL, threads=threads)
    return lr.shape[0] * lr.shape[2] * r * lr.shape[3] * r  # HR pixels processed


def time_oracle(wl, lr, dict_, coef, S, gamma, budget_s: float = 20.0):
    """Times the oracle on a bounded sample: a band of LR rows sized for roughly `budget_s` seconds."""
    import oracle
    probe_rows = max(1, min(wl.h, 8))
    t0 = time.perf_counter()
    px = oracle_step(oracle, wl, lr[:1], dict_, coef[:1], S, gamma, probe_rows)
    dt = time.perf_counter() - t0
    rate = px / dt
    rows = int(max(probe_rows, min(wl.h, budget_s * rate / (wl.W * wl.scale))))
    # when a whole frame takes less than the budget, the same band is repeated until about 14 s have been spent
    reps = int(max(1, min(64, (0.7 * budget_s * rate) // max(1, rows * wl.scale * wl.W))))
    t0 = time.perf_counter()
    px = 0
    for _ in range(reps):
        px += oracle_step(oracle, wl, lr[:1], dict_, coef[:1], S, gamma, rows)
    dt = time.perf_counter() - t0
    return {"value": px / dt / 1e6, "unit": METRIC, "cores": oracle.max_threads(), "kind": "oracle",
            "sample": f"top {rows} of {wl.h} LR rows of one frame, {reps} times ({px} HR pixels), all six paths of a "
                      f"step, {dt:.2f} s of fp64 CPU work"}


def run_reference(args, wl):
    """The reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    import numpy as np
    import sr_inputs
    one = sr_inputs.Workload(wl.name, 1, wl.c, wl.h, wl.w, wl.scale, wl.D, wl.k, wl.coef_dtype, wl.s)
    lr, dict_, coef = sr_inputs.make_inputs(one)
    S = np.arange(0, wl.D, max(1, wl.D // wl.s), dtype=np.uint8)[: wl.s]
    gamma = np.linspace(0.75, 1.25, wl.s).astype(np.float32)
    # size a step so that warmup + steps end within a few minutes
    t0 = time.perf_counter()
    px = oracle_step(oracle, one, lr, dict_, coef, S, gamma, 4)
    rate = px / (time.perf_counter() - t0)
    budget = 120.0 / max(1, args.steps + args.warmup)
    rows = int(max(1, min(wl.h, budget * rate / (wl.W * wl.scale))))
    for _ in range(args.warmup):
        oracle_step(oracle, one, lr, dict_, coef, S, gamma, rows)
    t0 = time.perf_counter()
    px = 0
    for _ in range(args.steps):
        px += oracle_step(oracle, one, lr, dict_, coef, S, gamma, rows)
    dt = time.perf_counter() - t0
    value = px / dt / 1e6
    sample = f"top {rows} of {wl.h} LR rows of one frame per step, all six paths"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "MP/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl),
        "cpu_baseline": {"value": value, "unit": "MP/s", "cores": oracle.max_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "MP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def workload_config(wl):
    return {"workload": f"{wl.name}: LR {wl.n}x{wl.c}x{wl.h}x{wl.w} fp32, x{wl.scale} -> {wl.H}x{wl.W}, D={wl.D} atoms "
                        f"of {wl.k}x{wl.k}, coefficients {wl.coef_dtype} [n][D][H][W], top-s s={wl.s}",
            "paths_per_step": list(PATHS),
            "l2": "coefficient tensor per frame is larger than the 126 MB L2 and three buffer sets rotate between steps"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--workload", default="cfg1")
    ap.add_argument("--paths", default=",".join(PATHS), help="comma-separated subset of the step's paths (profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    active = tuple(p for p in PATHS if p in args.paths.split(","))
    if "compact" in active and "select" not in active:
        active = tuple(p for p in PATHS if p in active or p == "select")   # compact consumes select's outputs

    import sr_inputs
    wl = sr_inputs.CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
        return

    import numpy as np
    import torch
    import paper_2303_08999_b200 as sr

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    sr.load_library()

    # ---- inputs: every rank owns its own frames (seed offset by rank); three rotating buffer sets
    seed = rank_seed(sr_inputs.BASE_SEED, rank)
    lr, dict_, coef = sr_inputs.make_inputs(wl, seed)
    S = np.arange(0, wl.D, max(1, wl.D // wl.s), dtype=np.uint8)[: wl.s]
    gamma = np.linspace(0.75, 1.25, wl.s).astype(np.float32)
    nsets = 3
    h_lr = torch.from_numpy(lr).pin_memory()
    h_coef = torch.from_numpy(coef).pin_memory()
    d_dict, d_S, d_gamma = (torch.from_numpy(a).cuda() for a in (dict_, S, gamma))
    sets = []
    for _ in range(nsets):
        sets.append({"lr": h_lr.cuda(non_blocking=True), "coef": h_coef.cuda(non_blocking=True)})
    shape_out = (wl.n, wl.c, wl.H, wl.W)
    outs = {p: torch.empty(shape_out, dtype=torch.float32, device="cuda") for p in ("bicubic", "dense", "compact", "fused", "global")}
    idx = torch.empty((wl.n, wl.s, wl.H, wl.W), dtype=torch.uint8, device="cuda")
    sel = torch.empty((wl.n, wl.s, wl.H, wl.W), dtype=h_coef.dtype, device="cuda")
    flags = sr.SR_CLAMP01
    r, k, s = wl.scale, wl.k, wl.s
    torch.cuda.synchronize()

    def step(bufs, events=None, outs=outs, only=None):
        """One step. With `events`, a CUDA event is recorded before and after every call (`only`: around that path's
        call alone); each record costs about 3 us of stream time, so the headline region records as few as it can."""
        def mark(*paths):
            if events is not None and (only is None or only in paths):
                e = torch.cuda.Event(enable_timing=True)
                e.record()
                events.append(e)
        mark("bicubic")
        if "bicubic" in active:
            sr.sr_bicubic_upsample(bufs["lr"], r, out=outs["bicubic"])
        mark("bicubic", "dense")
        if "dense" in active:
            sr.sr_dict_regress_dense(bufs["lr"], bufs["coef"], d_dict, r, k, flags, out=outs["dense"])
        mark("dense", "select")
        if "select" in active:
            sr.sr_dict_select(bufs["coef"], s, idx=idx, sel=sel)
        mark("select", "compact")
        if "compact" in active:
            sr.sr_dict_regress_selected(bufs["lr"], sel, idx, None, d_dict, r, k, s, flags | sr.SR_COEF_COMPACT, out=outs["compact"])
        mark("compact", "fused")
        if "fused" in active:
            sr.sr_dict_regress_selected(bufs["lr"], bufs["coef"], None, None, d_dict, r, k, s, flags, out=outs["fused"])
        mark("fused", "global")
        if "global" in active:
            sr.sr_dict_regress_selected(bufs["lr"], bufs["coef"], d_S, d_gamma, d_dict, r, k, s, flags | sr.SR_IDX_GLOBAL, out=outs["global"])
        mark("global")

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:
        pass
    sampler = ClockSampler(uuid) if rank == 0 else None
    if sampler:
        sampler.wait_first_sample()
    for i in range(args.warmup):
        step(sets[i % nsets])
    barrier()

    # ---- per-path pass (not the headline): the same K steps with an event between every call. It gives every path's
    # time and names the slowest one, whose kernel the roofline object describes.
    pass_events = []
    for i in range(args.steps):
        step(sets[i % nsets], pass_events)
    barrier()
    per_path_ms = {}
    per = len(PATHS) + 1
    for j, p in enumerate(PATHS):
        ts = [pass_events[i * per + j].elapsed_time(pass_events[i * per + j + 1]) for i in range(args.steps)]
        per_path_ms[p] = sum(ts) / len(ts)
    dominant_now = max(active, key=lambda p: per_path_ms[p])

    # ---- timed region: exactly K steps; events only around the slowest path's call (its duration for the roofline)
    launches0 = sr.sr_launch_count()
    events = []
    barrier()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    t_start.record()
    for i in range(args.steps):
        step(sets[i % nsets], events, only=dominant_now)
    t_end.record()
    barrier()
    wall1 = time.time()
    elapsed_ms = t_start.elapsed_time(t_end)
    launches = sr.sr_launch_count() - launches0
    clocks = sampler.stop(wall0, wall1) if sampler else None
    if sr.sr_device_status() != 0:
        raise SystemExit("device status word reports an expired wait")
    elapsed_ms = max_over_ranks(elapsed_ms, dist, "cuda")
    assert len(events) == 2 * args.steps
    ts = [events[2 * i].elapsed_time(events[2 * i + 1]) for i in range(args.steps)]
    per_path_ms[dominant_now] = sum(ts) / len(ts)               # the roofline kernel's time comes from the timed region

    # ---- end to end through the public API with host buffers: pinned H2D of the step's inputs, D2H of its results
    e2e = None
    if not args.no_e2e:
        # Two figures.  `value`: a stream of frames through HostPipeline (step i+1's inputs travel while step i's
        # results do; every step still copies all its inputs in and all its results out inside the timed region).
        # `serial_value`: one step at a time on one stream, copy in -> kernels -> copy out.
        from paper_2303_08999_b200.hostpipe import HostPipeline
        h_out = {p: torch.empty(shape_out, dtype=torch.float32).pin_memory() for p in outs}
        e2e_steps = max(3, min(args.steps, 10))
        host_in = {"lr": h_lr, "coef": h_coef}
        pipe = HostPipeline({"lr": (tuple(h_lr.shape), h_lr.dtype), "coef": (tuple(h_coef.shape), h_coef.dtype)},
                            {p: (shape_out, torch.float32) for p in outs}, depth=2)

        def timed(fn, after):
            fn()
            after()
            barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(e2e_steps):
                fn()
            after()
            b.record()
            barrier()
            return max_over_ranks(a.elapsed_time(b), dist, "cuda")

        def serial_step():
            bufs = sets[0]
            bufs["lr"].copy_(h_lr, non_blocking=True)
            bufs["coef"].copy_(h_coef, non_blocking=True)
            step(bufs)
            for p in outs:
                h_out[p].copy_(outs[p], non_blocking=True)

        ms_serial = timed(serial_step, lambda: None)
        ms_pipe = timed(lambda: pipe.submit(host_in, h_out, lambda i, o: step(i, None, o)), pipe.drain)
        if "dense" in active and not torch.equal(h_out["dense"], outs["dense"].cpu()):
            raise SystemExit("pipelined end-to-end result differs from the device-resident one")
        e2e = {"value": whole_job_value(world, wl.npix, e2e_steps, ms_pipe), "unit": "MP/s",
               "h2d_bytes_per_step": h_lr.numel() * 4 + h_coef.numel() * h_coef.element_size(),
               "d2h_bytes_per_step": sum(o.numel() * 4 for o in outs.values()), "steps": e2e_steps,
               "how": "HostPipeline, depth 2: copy-in, kernels and copy-out on three streams",
               "serial_value": whole_job_value(world, wl.npix, e2e_steps, ms_serial)}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = load_peaks()
    paths = {}
    for p in active:
        by = algorithmic_bytes_per_pixel(wl, p) * wl.npix
        gbs = by / (per_path_ms[p] * 1e-3) / 1e9
        paths[p] = {"ms": per_path_ms[p], "mp_per_s": wl.npix / (per_path_ms[p] * 1e-3) / 1e6,
                    "frames_per_s": wl.n / (per_path_ms[p] * 1e-3), "algorithmic_bytes": by, "achieved_gbs": gbs,
                    "frac_of_hbm": gbs / peak}
    dominant = dominant_now
    roofline = path_roofline(wl, dominant, per_path_ms[dominant], peak, peak_kind, NCU_TRAFFIC_BYTES_PER_PIXEL.get(dominant))
    for p in active:
        paths[p]["roofline"] = path_roofline(wl, p, per_path_ms[p], peak, peak_kind, NCU_TRAFFIC_BYTES_PER_PIXEL.get(p))

    cpu = None
    if not args.no_cpu_baseline:
        cpu = time_oracle(wl, lr, dict_, coef, S, gamma)

    line = {
        "metric": METRIC, "value": whole_job_value(world, wl.npix, args.steps, elapsed_ms), "unit": "MP/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32 accumulate, f16 coefficients"
        if wl.coef_dtype == "f16" else "f32", "data": "synthetic", "config": dict(workload_config(wl), paths_per_step=list(active)),
        "gpu_launches": int(launches), "clocks": clocks, "e2e": e2e, "roofline": roofline, "cpu_baseline": cpu,
        "paths": paths,
        "paths_timing": "pass of K steps with an event between every call, before the timed region; the roofline "
                        "kernel's time is from the events inside the timed region",
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
