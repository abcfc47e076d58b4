#!/usr/bin/env python
"""Benchmark of the dictionary-regression hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg0|cfg1|cfg2|cfg3|cfg4|producer|extras]

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

Workloads: cfg1 (the default; cfg2 is the same frame) prints the one JSON line of the benchmark contract. cfg0 (fp32
coefficients, 128 x 128 output) and cfg3 (batch of four 4K frames) print one line of the same form. cfg4 is the shape
sweep (LR 360 x 640, scale in {2,3,4}, D in {16,32,72,128}, k in {3,5,7}, s in {4,8,16}): one line per point and s, each
with the per-path times and roofline fractions, the clocks seen during its timed region and the oracle timed on a
small sample (`--points r3_D72_k5` restricts the sweep, `--s 8` its list lengths). Every path's roofline is the slowest of its bytes at the
measured HBM bandwidth, its selection-network operations at the measured integer max/min rate and its multiply-adds
at the measured fp32 rate (both rates are measured at start-up by the library's probe kernels).
`--workload producer` times the regression fused with the last layer of the coefficient network (sr_producer_regress, one
call per step on the cfg1 frame, features [n][h][w][32] binary16, 3x3 convolution): its roofline is the folded
convolution's tensor-core work against the measured dense bf16 rate. `--workload extras` prints three more lines (output and
up-sampling variants, the selection search, the tile-shape search); see run_extras.
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


# DRAM bytes per HR pixel seen by ncu (dram__bytes_read.sum + dram__bytes_write.sum) for each path's kernel on the
# 1080p x4 frame (cfg1 / cfg2 only; figures and commands are in profiles/dram_traffic_cfg1.md). Figures below a path's
# algorithmic bytes: the output (24.9 MB frame, 49.8 MB of index + value planes) is still in the 126 MB L2 when the kernel ends.
NCU_TRAFFIC_BYTES_PER_PIXEL = {"bicubic": 0.8, "dense": 154.2, "select": 163.5, "compact": 25.5, "fused": 154.1, "global": 16.8}


def selection_network_ops_per_pixel(path: str, D: int, s: int):
    """Integer / packed max-min lane operations per HR pixel of the selection networks (csrc/sr_select.cu and the select
    role of csrc/sr_umma_impl.inc): per group of eight planes a 19-exchange sort and a merge into the running list
    (8 max + a 12-exchange bitonic merge for a list of 8; 8 max + 32 exchanges for a list of 16). The stand-alone kernel
    works on 32-bit keys, one pixel per lane operation; the fused kernel on packed binary16 pairs, two pixels per lane
    operation, plus 36 magnitude / logic and 40 address operations per 72 planes. These are the networks' own
    operations, all counted at the integer max/min rate: building the keys and the tails add to them on the same pipe
    (overhead, not part of the bound), and the stand-alone kernel runs one compare-exchange in five on the FMA pipe
    instead (five exact fp32 operations each), which is how it can come closer to this bound than the ALU pipe alone
    would let it."""
    if s > 16 or path not in ("select", "fused"):
        return 0.0
    if path == "select":
        # list of 4, 8 or 16 keys; groups of as many planes: sort (5 / 19 / 70 exchanges) + S max + merge (4 / 12 / 32 exchanges)
        S, per_group = (4, 22.0) if s <= 4 else ((8, 70.0) if s <= 8 else (16, 220.0))
        return per_group * ((D + S - 1) // S)
    # fused: groups of eight planes against a list of 8 (s <= 8) or 16, two pixels per lane operation
    per_group = 70.0 if s <= 8 else 110.0
    return (per_group / 2 + 8.4) * ((D + 7) // 8)


def fma_macs_per_pixel(wl, path: str):
    """fp32 multiply-adds per HR pixel of the paths that run on the FMA pipe, or are bounded by it because their atoms are too few for a tensor-core contraction:
    the small subset and compact forms (s k^2 + c k^2: assemble the filter from s atoms, then filter), and every
    regression with fp32 coefficients (general kernel: D k^2 + c k^2)."""
    kk = wl.k * wl.k
    if wl.coef_dtype == "f32" and path in ("dense", "fused", "compact", "global"):
        atoms = wl.D if path == "dense" else wl.s
        return float(atoms * kk + wl.c * kk)
    if path in ("compact", "global") and wl.s <= 8:
        return float(wl.s * kk + wl.c * kk)
    return 0.0


def path_roofline(wl, path: str, ms: float, peaks: dict, traffic_bytes_per_pixel):
    """Roofline entry of one path: the slowest of its bytes at HBM bandwidth, its selection operations at the integer
    max/min rate and its multiply-adds at the fp32 rate; `frac` = that time / the measured time."""
    by = algorithmic_bytes_per_pixel(wl, path) * wl.npix
    ops = selection_network_ops_per_pixel(path, wl.D, wl.s) * wl.npix
    macs = fma_macs_per_pixel(wl, path) * wl.npix
    t = {"hbm": by / (peaks["hbm_gbs"] * 1e9), "alu": ops / peaks["alu_ops"], "fma": macs / peaks["fma_ops"]}
    bound = max(t, key=lambda k: t[k])
    traffic = None if traffic_bytes_per_pixel is None else traffic_bytes_per_pixel * wl.npix
    sec = ms * 1e-3
    if bound == "hbm":
        out = {"bound": "hbm", "achieved": by / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s", "peak_kind": f"of {peaks['hbm_kind']}"}
    elif bound == "alu":
        out = {"bound": "alu", "achieved": ops / sec / 1e9, "peak": peaks["alu_ops"] / 1e9, "unit": "Gop/s (max/min lanes)",
               "peak_kind": "measured at start-up by sr_probe_rate(0)"}
    else:
        out = {"bound": "fma", "achieved": macs / sec / 1e9, "peak": peaks["fma_ops"] / 1e9, "unit": "GMAC/s (fp32)",
               "peak_kind": "measured at start-up by sr_probe_rate(1)"}
    out.update({"kernel": path, "frac": out["achieved"] / out["peak"], "traffic": traffic, "roofline_us": t[bound] * 1e6,
                "hbm_frac": by / sec / 1e9 / peaks["hbm_gbs"]})
    return out


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


def run_reference_producer(args, wl):
    """Reference arm of `--workload producer`: the oracle's producer + regression on a band of LR rows per step."""
    import oracle
    import sr_inputs
    one = sr_inputs.Workload(wl.name, 1, wl.c, wl.h, wl.w, wl.scale, wl.D, wl.k, wl.coef_dtype, wl.s)
    lr, dict_ = sr_inputs.make_lr(one), sr_inputs.make_dictionary(wl.D, wl.k)
    feat, wconv, bias = sr_inputs.make_producer(one, PRODUCER_CIN, PRODUCER_KC)
    call = lambda rows: oracle.producer_regress(lr[:, :, :rows].copy(), feat[:, :rows].copy(), wconv, bias, dict_, wl.scale, wl.k,
                                                flags=oracle.CLAMP01)
    t0 = time.perf_counter()
    call(4)
    rate = 4 / (time.perf_counter() - t0)
    rows = int(max(1, min(wl.h, 120.0 / max(1, args.steps + args.warmup) * rate)))
    for _ in range(args.warmup):
        call(rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        call(rows)
    dt = time.perf_counter() - t0
    value = args.steps * rows * wl.scale * wl.W / dt / 1e6
    sample = f"top {rows} of {wl.h} LR rows of one frame per step, producer + regression"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "MP/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": "producer (cfg1 frame, 32 feature channels, 3x3 convolution)"},
        "cpu_baseline": {"value": value, "unit": "MP/s", "cores": oracle.max_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "MP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def run_reference(args, wl, producer: bool = False):
    """The reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    if producer:
        return run_reference_producer(args, wl)
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
        "config": workload_config(wl, 1),
        "cpu_baseline": {"value": value, "unit": "MP/s", "cores": oracle.max_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "MP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def workload_config(wl, nsets: int):
    return {"workload": f"{wl.name}: LR {wl.n}x{wl.c}x{wl.h}x{wl.w} fp32, x{wl.scale} -> {wl.H}x{wl.W}, D={wl.D} atoms "
                        f"of {wl.k}x{wl.k}, coefficients {wl.coef_dtype} [n][D][H][W], top-s s={wl.s}",
            "paths_per_step": list(PATHS),
            "l2": f"{nsets} coefficient buffer sets rotate between steps; together they are larger than twice the 126 MB L2"}


def rotating_sets(coef_bytes: int) -> int:
    """Buffer sets to rotate through so that no coefficient read is served by the L2 (126 MB) of an earlier step."""
    need = 2 * 126 * 1024 * 1024
    return int(max(3, min(96, -(-need // max(1, coef_bytes)))))


def measure_peaks(sr):
    hbm, kind = load_peaks()
    # fp32 multiply-adds: the better of the scalar and the packed (two per lane and instruction) issue rates
    return {"hbm_gbs": hbm, "hbm_kind": kind, "alu_ops": sr.sr_probe_rate(0), "fma_ops": max(sr.sr_probe_rate(1), sr.sr_probe_rate(2))}


def run_workload(wl, args, active, peaks, dist, rank, world, local_rank, steps: int, warmup: int, with_e2e: bool, cpu_budget_s: float):
    """Runs one workload on this rank and returns rank 0's JSON line (None on the other ranks)."""
    import numpy as np
    import torch
    import paper_2303_08999_b200 as sr
    import sr_inputs

    # ---- inputs: every rank owns its own frames (seed offset by rank); rotating buffer sets
    seed = rank_seed(sr_inputs.BASE_SEED, rank)
    lr, dict_, coef = sr_inputs.make_inputs(wl, seed)
    S = np.arange(0, wl.D, max(1, wl.D // wl.s), dtype=np.uint8)[: wl.s]
    gamma = np.linspace(0.75, 1.25, wl.s).astype(np.float32)
    nsets = rotating_sets(coef.nbytes)
    h_lr = torch.from_numpy(lr).pin_memory() if with_e2e else torch.from_numpy(lr)
    h_coef = torch.from_numpy(coef).pin_memory() if with_e2e else torch.from_numpy(coef)
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
    for i in range(warmup):
        step(sets[i % nsets])
    barrier()

    # ---- per-path pass (not the headline): the same K steps with an event between every call. It gives every path's
    # time and names the slowest one, whose kernel the roofline object describes.
    pass_events = []
    for i in range(steps):
        step(sets[i % nsets], pass_events)
    barrier()
    per_path_ms = {}
    per = len(PATHS) + 1
    for j, p in enumerate(PATHS):
        ts = [pass_events[i * per + j].elapsed_time(pass_events[i * per + j + 1]) for i in range(steps)]
        per_path_ms[p] = sum(ts) / len(ts)
    dominant_now = max(active, key=lambda p: per_path_ms[p])

    # ---- timed region: exactly K steps; events only around the slowest path's call (its duration for the roofline)
    launches0 = sr.sr_launch_count()
    events = []
    barrier()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    t_start.record()
    for i in range(steps):
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
    assert len(events) == 2 * steps
    ts = [events[2 * i].elapsed_time(events[2 * i + 1]) for i in range(steps)]
    per_path_ms[dominant_now] = sum(ts) / len(ts)               # the roofline kernel's time comes from the timed region

    # ---- end to end through the public API with host buffers: pinned H2D of the step's inputs, D2H of its results
    e2e = None
    if with_e2e:
        # Two figures.  `value`: a stream of frames through HostPipeline (step i+1's inputs travel while step i's
        # results do; every step still copies all its inputs in and all its results out inside the timed region).
        # `serial_value`: one step at a time on one stream, copy in -> kernels -> copy out.
        from paper_2303_08999_b200.hostpipe import HostPipeline
        h_out = {p: torch.empty(shape_out, dtype=torch.float32).pin_memory() for p in outs}
        e2e_steps = max(3, min(steps, 10))
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

    del sets, outs, idx, sel
    torch.cuda.empty_cache()
    if rank != 0:
        return None

    traffic = NCU_TRAFFIC_BYTES_PER_PIXEL if wl.name in ("cfg1", "cfg2") else {}
    paths = {}
    for p in active:
        by = algorithmic_bytes_per_pixel(wl, p) * wl.npix
        gbs = by / (per_path_ms[p] * 1e-3) / 1e9
        paths[p] = {"ms": per_path_ms[p], "mp_per_s": wl.npix / (per_path_ms[p] * 1e-3) / 1e6,
                    "frames_per_s": wl.n / (per_path_ms[p] * 1e-3), "algorithmic_bytes": by, "achieved_gbs": gbs,
                    "frac_of_hbm": gbs / peaks["hbm_gbs"],
                    "roofline": path_roofline(wl, p, per_path_ms[p], peaks, traffic.get(p))}
    roofline = path_roofline(wl, dominant_now, per_path_ms[dominant_now], peaks, traffic.get(dominant_now))

    cpu = None
    if cpu_budget_s > 0:
        cpu = time_oracle(wl, lr, dict_, coef, S, gamma, budget_s=cpu_budget_s)

    return {
        "metric": METRIC, "value": whole_job_value(world, wl.npix, steps, elapsed_ms), "unit": "MP/s",
        "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": elapsed_ms / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32 accumulate, f16 coefficients"
        if wl.coef_dtype == "f16" else "f32", "data": "synthetic", "config": dict(workload_config(wl, nsets), paths_per_step=list(active)),
        "gpu_launches": int(launches), "clocks": clocks, "e2e": e2e, "roofline": roofline, "cpu_baseline": cpu,
        "paths": paths,
        "peaks": {"hbm_gbs": peaks["hbm_gbs"], "hbm": f"of {peaks['hbm_kind']}", "int_maxmin_gops": peaks["alu_ops"] / 1e9,
                  "fp32_fma_gmacs": peaks["fma_ops"] / 1e9, "how": "HBM: MEASURED_PEAKS.json; pipes: sr_probe_rate at start-up (fp32: the better of scalar and packed multiply-add)"},
        "paths_timing": "pass of K steps with an event between every call, before the timed region; the roofline "
                        "kernel's time is from the events inside the timed region",
    }


PRODUCER_CIN, PRODUCER_KC = 32, 3


def producer_flops(wl, cin: int, kc: int) -> float:
    """Tensor-core work of the fused last layer per launch: the folded convolution, 2 x LR pixels x (kc^2 cin) x
    (r^2 k^2) (the bias K-step and the padding columns are not counted)."""
    return 2.0 * wl.n * wl.h * wl.w * (kc * kc * cin) * (wl.scale ** 2 * wl.k ** 2)


def producer_bytes(wl, cin: int) -> float:
    """Bytes that must cross HBM per launch: feature map and LR frame read once, output written once."""
    return float(wl.n * wl.h * wl.w * (cin * 2 + 4 * wl.c) + wl.npix * 4 * wl.c)


def time_oracle_producer(wl, lr, feat, wconv, bias, dict_, budget_s: float):
    import oracle
    rows = 4
    t0 = time.perf_counter()
    oracle.producer_regress(lr[:1, :, :rows], feat[:1, :rows], wconv, bias, dict_, wl.scale, wl.k, flags=oracle.CLAMP01)
    rate = rows / (time.perf_counter() - t0)
    rows = int(max(4, min(wl.h, budget_s * rate)))
    t0 = time.perf_counter()
    oracle.producer_regress(lr[:1, :, :rows].copy(), feat[:1, :rows].copy(), wconv, bias, dict_, wl.scale, wl.k, flags=oracle.CLAMP01)
    dt = time.perf_counter() - t0
    px = rows * wl.scale * wl.W
    return {"value": px / dt / 1e6, "unit": "MP/s", "cores": oracle.max_threads(), "kind": "oracle",
            "sample": f"top {rows} of {wl.h} LR rows of one frame ({px} HR pixels), producer + regression, {dt:.2f} s of fp64 CPU work"}


def run_producer(wl, args, dist, rank, world, local_rank, steps: int, warmup: int):
    """`--workload producer`: the regression fused with the last convolution + pixel-shuffle of the coefficient network
    (sr_producer_regress) on the 1080p x4 frame; one step = one call. The dictionary is folded into the layer's
    weights once, outside the timed region (it depends on the network and the dictionary, not on the frame)."""
    import numpy as np
    import torch
    import paper_2303_08999_b200 as sr
    import sr_inputs

    cin, kc = PRODUCER_CIN, PRODUCER_KC
    seed = rank_seed(sr_inputs.BASE_SEED, rank)
    lr = sr_inputs.make_lr(wl, seed)
    dict_ = sr_inputs.make_dictionary(wl.D, wl.k, seed)
    feat, wconv, bias = sr_inputs.make_producer(wl, cin, kc, seed)
    h_lr, h_feat = torch.from_numpy(lr).pin_memory(), torch.from_numpy(feat).pin_memory()
    folded = sr.sr_producer_fold(*(torch.from_numpy(a).cuda() for a in (wconv, bias, dict_)), wl.scale, wl.k)
    shape_out = (wl.n, wl.c, wl.H, wl.W)
    per_set = feat.nbytes + lr.nbytes + 4 * wl.n * wl.c * wl.H * wl.W
    nsets = int(max(3, min(96, -(-2 * 126 * 1024 * 1024 // per_set))))
    sets = [{"lr": h_lr.cuda(), "feat": h_feat.cuda(), "out": torch.empty(shape_out, dtype=torch.float32, device="cuda")}
            for _ in range(nsets)]
    flags = sr.SR_CLAMP01

    def step(b, out=None):
        sr.sr_producer_regress(b["lr"], b["feat"], folded, wl.scale, wl.k, wl.D, kc, flags, out=b["out"] if out is None else out)

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
    for i in range(warmup):
        step(sets[i % nsets])
    barrier()
    # the kernel's own duration: an event on both sides of every launch (not the headline)
    evs = []
    for i in range(steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); step(sets[i % nsets]); b.record()
        evs.append((a, b))
    barrier()
    kernel_ms = sum(a.elapsed_time(b) for a, b in evs) / steps
    launches0 = sr.sr_launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    wall0 = time.time()
    t0.record()
    for i in range(steps):
        step(sets[i % nsets])
    t1.record()
    barrier()
    wall1 = time.time()
    elapsed_ms = max_over_ranks(t0.elapsed_time(t1), dist, "cuda")
    launches = sr.sr_launch_count() - launches0
    clocks = sampler.stop(wall0, wall1) if sampler else None
    if sr.sr_device_status() != 0:
        raise SystemExit("device status word reports an expired wait")

    # end to end: pinned host -> device copies of the LR frame and the feature map, device -> host copy of the result
    e2e = None
    if not args.no_e2e:
        from paper_2303_08999_b200.hostpipe import HostPipeline
        h_out = {"out": torch.empty(shape_out, dtype=torch.float32).pin_memory()}
        pipe = HostPipeline({"lr": (tuple(h_lr.shape), h_lr.dtype), "feat": (tuple(h_feat.shape), h_feat.dtype)},
                            {"out": (shape_out, torch.float32)}, depth=2)
        e2e_steps = max(3, min(steps, 20))
        fn = lambda: pipe.submit({"lr": h_lr, "feat": h_feat}, h_out, lambda i, o: step(i, o["out"]))
        fn(); pipe.drain(); barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(e2e_steps):
            fn()
        pipe.drain()
        b.record()
        barrier()
        ms = max_over_ranks(a.elapsed_time(b), dist, "cuda")
        e2e = {"value": whole_job_value(world, wl.npix, e2e_steps, ms), "unit": "MP/s",
               "h2d_bytes_per_step": lr.nbytes + feat.nbytes, "d2h_bytes_per_step": 4 * wl.n * wl.c * wl.H * wl.W,
               "steps": e2e_steps, "how": "HostPipeline, depth 2: copy-in, kernel and copy-out on three streams"}
    if rank != 0:
        return None
    tf_peak, tf_kind = load_tensor_peak()
    fl = producer_flops(wl, cin, kc)
    by = producer_bytes(wl, cin)
    sec = kernel_ms * 1e-3
    roofline = {"bound": "tensor", "kernel": "producer_regress_kernel", "achieved": fl / sec / 1e12, "peak": tf_peak, "unit": "TFLOP/s",
                "frac": fl / sec / 1e12 / tf_peak, "peak_kind": f"of {tf_kind} (dense bf16 burst; binary16 runs at the same nominal rate)",
                "traffic": None, "roofline_us": fl / (tf_peak * 1e12) * 1e6, "kernel_us": kernel_ms * 1e3,
                "hbm_bytes": by, "hbm_frac": by / sec / 1e9 / load_peaks()[0],
                "bytes_a_separate_coefficient_tensor_would_add": 2.0 * wl.D * 2 * wl.npix}
    cpu = None if args.no_cpu_baseline else time_oracle_producer(wl, lr, feat, wconv, bias, dict_, 15.0)
    return {
        "metric": METRIC, "value": whole_job_value(world, wl.npix, steps, elapsed_ms), "unit": "MP/s", "n_gpus": world,
        "steps": steps, "warmup": warmup, "ms_per_step": elapsed_ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16 operands, f32 accumulate", "data": "synthetic",
        "config": {"workload": f"producer: LR {wl.n}x{wl.c}x{wl.h}x{wl.w} fp32 + features [n][h][w][{cin}] f16, last layer "
                               f"{kc}x{kc} conv -> {wl.D}x{wl.scale}^2 channels + pixel-shuffle x{wl.scale}, D={wl.D} atoms of "
                               f"{wl.k}x{wl.k}, folded; one sr_producer_regress call per step",
                   "l2": f"{nsets} sets of (features, LR frame, output) rotate between steps; together larger than twice the 126 MB L2"},
        "gpu_launches": int(launches), "clocks": clocks, "e2e": e2e, "roofline": roofline, "cpu_baseline": cpu,
    }


def run_extras(wl, args, peaks):
    """`--workload extras`: the rows beyond the benchmark step, on the cfg1 frame, one JSON line each (CUDA events, median
    of `--steps` launches after 3 warm-up launches, 256 MB written between launches to flush the L2):
      variants   dense regression with binary16 / 8-bit output, bilinear up-sampling, luma-only
      selection  Gram statistics of the selection search (every pixel; 100 000 sampled pixels) and Algorithm 1 on them
      tune       the tile-shape search on three shapes: default launch shape against the best found"""
    import numpy as np
    import torch
    import paper_2303_08999_b200 as sr
    import sr_inputs
    from dataclasses import replace

    steps = max(5, min(args.steps, 50))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def timed(fn, reps=steps):
        for _ in range(3):
            fn()
        ts = []
        for i in range(reps):
            flush.fill_(i & 255)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) * 1e3)
        return statistics.median(ts), min(ts)

    lr, dict_, coef = sr_inputs.make_inputs(wl)
    dlr, ddi, dco = (torch.from_numpy(a).cuda() for a in (lr, dict_, coef))
    r, k, s, D = wl.scale, wl.k, wl.s, wl.D
    base = {"workload": f"{wl.name}: LR {wl.n}x{wl.c}x{wl.h}x{wl.w}, x{r}, D={D}, k={k}", "steps": steps, "unit": "us", "data": "synthetic"}
    # ---- output and up-sampling variants of the dense call
    out = {}
    for name, fl in (("fp32 output", 0), ("binary16 output", sr.SR_OUT_F16), ("8-bit output", sr.SR_OUT_U8),
                     ("bilinear up-sampling", sr.SR_UPSAMPLE_BILINEAR), ("luma-only (one-channel regression + chroma)", sr.SR_LUMA_ONLY)):
        med, mn = timed(lambda: sr.sr_dict_regress_dense(dlr, dco, ddi, r, k, sr.SR_CLAMP01 | fl))
        obytes = {0: 4, sr.SR_OUT_F16: 2, sr.SR_OUT_U8: 1}.get(fl, 4) * wl.c
        by = (D * 2 + obytes + 4 * wl.c / r ** 2) * wl.npix
        out[name] = {"median_us": med, "min_us": mn, "algorithmic_bytes": by, "frac_of_hbm": by / (med * 1e-6) / 1e9 / peaks["hbm_gbs"]}
    print(json.dumps(dict(base, extra="variants of sr_dict_regress_dense", results=out)), flush=True)
    # ---- selection search: Gram statistics + Algorithm 1
    S = np.arange(0, D, max(1, D // s), dtype=np.uint8)[:s]
    gamma = np.linspace(0.75, 1.25, s).astype(np.float32)
    target = sr.sr_dict_regress_selected(dlr, dco, torch.from_numpy(S).cuda(), torch.from_numpy(gamma).cuda(), ddi, r, k, s, sr.SR_IDX_GLOBAL)
    target = (target + 0.01 * torch.randn(target.shape, device="cuda", generator=torch.Generator("cuda").manual_seed(1))).contiguous()
    samples = torch.arange(0, wl.npix, max(1, wl.npix // 100000), device="cuda", dtype=torch.int64)[:100000].contiguous()
    macs_row = D * k * k + D * (D + 1) / 2 + D            # responses, upper triangle of z z^T, z h
    res = {}
    for name, smp, npx in (("every pixel", None, wl.npix), (f"{samples.numel()} sampled pixels", samples, samples.numel())):
        med, mn = timed(lambda: sr.sr_selection_gram(dlr, dco, ddi, target, smp, r, k), reps=max(3, steps // 5))
        macs = macs_row * npx * wl.c
        res["gram, " + name] = {"median_us": med, "min_us": mn, "fp32_macs": macs, "frac_of_fma": macs / (med * 1e-6) / peaks["fma_ops"]}
    G, b, hh = sr.sr_selection_gram(dlr, dco, ddi, target, samples, r, k)
    t0 = time.perf_counter()
    idx, gam, trace = sr.sr_selection_search(G, b, hh, samples.numel() * wl.c, s / D, 16.0 / D, 0.0, 1e-9)
    torch.cuda.synchronize()
    res["search (Algorithm 1, one warp, fp64)"] = {"wall_us": (time.perf_counter() - t0) * 1e6, "atoms_kept": int(idx.numel()),
                                                   "steps": int(trace.shape[0]), "found_the_planted_subset": bool(np.array_equal(idx.cpu().numpy(), S))}
    print(json.dumps(dict(base, extra="selection search (sr_selection_gram, sr_selection_search)", results=res)), flush=True)
    # ---- tile-shape search
    res = {}
    for name, w2 in (("cfg1 dense", wl), ("cfg4 r2 D16 k7 dense", replace(sr_inputs.CONFIGS["cfg4"], scale=2, D=16, k=7)),
                     ("cfg4 r3 D32 k5 dense", replace(sr_inputs.CONFIGS["cfg4"], scale=3, D=32, k=5))):
        l2, d2, c2 = (torch.from_numpy(a).cuda() for a in sr_inputs.make_inputs(w2))
        sr.sr_tune_reset()
        res[name] = sr.sr_tune_dense(l2, c2, d2, w2.scale, w2.k, sr.SR_CLAMP01, reps=10)
        S2 = torch.arange(0, w2.D, max(1, w2.D // 16), dtype=torch.uint8, device="cuda")[:16].contiguous()
        if S2.numel() == 16:
            res[name.replace("dense", "global subset s=16")] = sr.sr_tune_selected(l2, c2, S2, None, d2, w2.scale, w2.k, 16, sr.SR_CLAMP01 | sr.SR_IDX_GLOBAL, reps=10)
        del l2, d2, c2
    sr.sr_tune_reset()
    print(json.dumps(dict(base, extra="tile-shape search (sr_tune_dense, sr_tune_selected): default launch shape against the best of the candidates", results=res)), flush=True)


def load_tensor_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        if "bf16_tflops" in d:
            return float(d["bf16_tflops"]), "measured"
    return 1590.0, "fallback"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--workload", default="cfg1")
    ap.add_argument("--points", default="", help="cfg4 only: comma-separated substrings of point names, e.g. r3_D72_k5")
    ap.add_argument("--s", type=int, default=0, help="cfg4 only: keep one list length of the sweep's 4, 8, 16")
    ap.add_argument("--paths", default=",".join(PATHS), help="comma-separated subset of the step's paths (profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    sweep = args.workload == "cfg4"
    steps = args.steps if args.steps is not None else (20 if sweep else (30 if args.workload == "cfg3" else (3000 if args.workload == "producer" else 300)))
    warmup = args.warmup if args.warmup is not None else (3 if sweep or args.workload == "cfg3" else 10)
    if args.impl == "ours":
        warmup = max(warmup, 3)
    args.steps, args.warmup = steps, warmup
    active = tuple(p for p in PATHS if p in args.paths.split(","))
    if "compact" in active and "select" not in active:
        active = tuple(p for p in PATHS if p in active or p == "select")   # compact consumes select's outputs

    import sr_inputs
    from dataclasses import replace
    producer = args.workload == "producer"
    if producer or args.workload == "extras":
        wls = [sr_inputs.CONFIGS["cfg1"]]
    elif sweep:
        want = [w for w in args.points.split(",") if w]
        wls = [replace(p, s=s) for p in sr_inputs.cfg4_points() for s in (4, 8, 16)
               if s <= p.D and (not args.s or s == args.s) and (not want or any(w in p.name for w in want))]
    else:
        wls = [sr_inputs.CONFIGS[args.workload]]
    if args.impl == "reference":
        run_reference(args, wls[0] if producer else sr_inputs.CONFIGS[args.workload], producer)   # the sweep's reference arm times its anchor point
        return

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
    peaks = measure_peaks(sr)
    default_line = args.workload in ("cfg1", "cfg2")
    if args.workload == "extras":
        if rank == 0:
            run_extras(sr_inputs.CONFIGS["cfg1"], args, peaks)
        if dist is not None:
            dist.destroy_process_group()
        return
    for wl in wls:
        if producer:
            line = run_producer(wl, args, dist, rank, world, local_rank, steps, warmup)
            if line is not None:
                print(json.dumps(line), flush=True)
            continue
        line = run_workload(wl, args, active, peaks, dist, rank, world, local_rank, steps, warmup,
                            with_e2e=default_line and not args.no_e2e,
                            cpu_budget_s=0.0 if args.no_cpu_baseline else (1.0 if sweep else 20.0))
        if line is not None:
            print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
