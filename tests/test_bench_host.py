"""Host-side logic of bench.py that needs no GPU: the walk over the frame sequence, the whole-job
aggregation over ranks (checked with two gloo ranks on CPU), the reference arm."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_pingpong_walk_keeps_neighbouring_frames_adjacent():
    order = bench.pingpong(5)
    assert order == [0, 1, 2, 3, 4, 3, 2, 1]
    walk = [order[i % len(order)] for i in range(40)]
    assert all(abs(a - b) == 1 for a, b in zip(walk, walk[1:]))


def _rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(2.0 if rank == 0 else 5.0, world)          # rank 1 is the slow one
    out[rank] = (ms, bench.whole_job_rate(32, ms, world))
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_rank_and_the_whole_job():
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank, args=(2, 29531, out), nprocs=2, join=True)
        for r in (0, 1):
            ms, rate = out[r]
            assert ms == 5.0
            assert rate == 2 * 32 * 1e3 / 5.0


def test_reference_arm_prints_the_contract_line():
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "3", "--warmup", "1"],
                       capture_output=True, text=True, check=True)
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "frames/s" and line["metric"] == "frames_per_sec"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["value"] > 0
