"""The multi-rank logic of bench.py on CPU: two `gloo` ranks.

The path shards by images with no exchange step, so what there is to test is
the bookkeeping: every rank times its own replica, the reported time is the
slowest rank's, the value counts all ranks' images, and only rank 0 prints.
"""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.rank_info() == (rank, rank, world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, device="cpu")     # rank 1 is the slow one
    value = bench.whole_job_value(128, 4, world, ms)
    dist.barrier()
    out.put((rank, ms, value))
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_value():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in got:
        assert ms == 15.0                                   # the slowest rank's time, on every rank
        assert abs(value - 2 * 128 * 4 / 15e-3) < 1e-6      # all ranks' images over that time


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, device="cpu") == 3.5
    assert bench.whole_job_value(128, 10, 1, 20.0) == 128 * 10 / 20e-3


def test_reference_arm_prints_on_rank_0_only():
    """`--impl reference` under a 2-rank launch: rank 0 times the oracle and prints
    the JSON line, the other rank exits 0 without work."""
    lines = {}
    for rank in (0, 1):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2")
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                            "--gpus", "2", "--steps", "1", "--warmup", "0"],
                           env=env, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr
        lines[rank] = r.stdout.strip()
    assert lines[1] == ""
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["cores"] >= 1
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["unit"] == "images/s"


def test_gpus_flag_alone_starts_that_many_ranks():
    """`bench.py --gpus 2` called plainly (no launcher environment) starts two ranks itself; here
    with the step stubbed out and `gloo`, which is what runs without GPUs.  One JSON line comes
    back, from rank 0, for two ranks, with the slowest rank's time and both ranks' images."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "stub", "--gpus", "2",
                        "--steps", "4"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, r.stdout
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == 2 and rec["impl"] == "stub"
    assert abs(rec["ms_per_step"] - 15.0 / 4) < 1e-9
    assert abs(rec["value"] - 2 * 128 * 4 / 15e-3) < 1e-6
