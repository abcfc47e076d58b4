"""Shape sweep of the regression paths (the cfg4 benchmark configuration): LR 3x360x640, scale in {2,3,4},
D in {16,32,72,128}, k in {3,5,7}; dense and fused selective (s in {4,8,16}, skipped when s > D).

    python -m paper_2303_08999_b200.sweep [--hbm-gbs 6459] [--cfg3]

Prints one markdown row per point: device time (CUDA events, median of 10 after 3 warm-up launches, three rotating
coefficient buffers when they fit so that nothing stays in L2), HR MP/s and the fraction of the HBM roofline
(algorithmic bytes = coefficients read once + output written once + LR read once).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import paper_2303_08999_b200 as sr  # noqa: E402
import sr_inputs  # noqa: E402


def time_us(fn, n=10, warm=3):
    for i in range(warm):
        fn(i)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
    ev[0].record()
    for i in range(n):
        fn(i)
        ev[i + 1].record()
    torch.cuda.synchronize()
    return sorted(ev[i].elapsed_time(ev[i + 1]) * 1e3 for i in range(n))[n // 2]


def run_point(wl, hbm_gbs, s_values):
    lr, dict_, coef = sr_inputs.make_inputs(wl)
    dlr, ddi = torch.from_numpy(lr).cuda(), torch.from_numpy(dict_).cuda()
    nbuf = 3 if coef.nbytes * 3 < 8e9 else 1
    cos = [torch.from_numpy(coef).cuda() for _ in range(nbuf)]
    out = torch.empty((wl.n, wl.c, wl.H, wl.W), dtype=torch.float32, device="cuda")
    bytes_px = wl.D * 2 + 4 * wl.c + 4 * wl.c / wl.scale ** 2
    rows = []
    t = time_us(lambda i: sr.sr_dict_regress_dense(dlr, cos[i % nbuf], ddi, wl.scale, wl.k, sr.SR_CLAMP01, out=out))
    rows.append(("dense", "-", t))
    for s in s_values:
        if s > wl.D:
            continue
        t = time_us(lambda i: sr.sr_dict_regress_selected(dlr, cos[i % nbuf], None, None, ddi, wl.scale, wl.k, s,
                                                          sr.SR_CLAMP01, out=out))
        rows.append(("fused select", str(s), t))
    for path, s, t in rows:
        gbs = bytes_px * wl.npix / (t * 1e-6) / 1e9
        print(f"| {wl.name} | {wl.n}x{wl.H}x{wl.W} | {wl.scale} | {wl.D} | {wl.k} | {path} | {s} | {t:.1f} | "
              f"{wl.npix / t:.0f} | {gbs:.0f} | {gbs / hbm_gbs:.3f} |", flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--hbm-gbs", type=float, default=None)
    ap.add_argument("--cfg3", action="store_true", help="also run the 4-frame 4K batch")
    args = ap.parse_args()
    hbm = args.hbm_gbs
    if hbm is None:
        p = os.path.join(ROOT, "MEASURED_PEAKS.json")
        hbm = float(json.load(open(p))["hbm_gbs"]) if os.path.exists(p) else 6650.0
    print(f"HBM peak used: {hbm} GB/s")
    print("| workload | HR frame | scale | D | k | path | s | us | HR MP/s | GB/s (algorithmic) | frac of HBM |")
    print("|---|---|---|---|---|---|---|---|---|---|---|")
    for wl in sr_inputs.cfg4_points():
        run_point(wl, hbm, (4, 8, 16))
    if args.cfg3:
        run_point(sr_inputs.CONFIGS["cfg3"], hbm, (8,))
        run_point(sr_inputs.CONFIGS["cfg0"], hbm, ())


if __name__ == "__main__":
    main()
