"""The N > 1 path of the benchmark on CPU: two gloo ranks, no GPU.

The method has no exchange step, so ranks only differ in their seeds and only meet for a barrier and the
max-over-ranks of the device time. These tests run that host logic with world_size 2.
"""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, {root!r})
    import numpy as np
    import torch.distributed as dist
    import bench, sr_inputs
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    seed = bench.rank_seed(sr_inputs.BASE_SEED, rank)
    wl = sr_inputs.Workload("t", 1, 3, 4, 6, 2, D=8, k=3, coef_dtype="f16")
    lr = sr_inputs.make_lr(wl, seed)
    dist.barrier()
    ms = bench.max_over_ranks(10.0 * (rank + 1), dist)          # rank 1 is the slow one
    value = bench.whole_job_value(world, wl.npix, 5, ms)
    print(json.dumps({{"rank": rank, "ms": ms, "value": value, "checksum": float(lr.sum()), "seed": seed}}), flush=True)
    dist.destroy_process_group()
""")


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_agree_on_max_time_and_own_their_frames(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                                      text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(__import__("json").loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert outs[0]["ms"] == outs[1]["ms"] == 20.0                    # the slowest rank's time on every rank
    pixels = 8 * 12
    assert abs(outs[0]["value"] - 2 * pixels * 5 / 0.020 / 1e6) < 1e-9   # whole job: both ranks' pixels
    assert outs[0]["seed"] + 1 == outs[1]["seed"] and outs[0]["checksum"] != outs[1]["checksum"]


def test_single_process_helpers():
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_value(1, 1_000_000, 10, 1000.0) == 10.0


def test_reference_arm_runs_on_rank_zero_only(tmp_path):
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
                          "--workload", "cfg0"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
