"""Host-side logic of the multi-GPU benchmark path, run as two gloo ranks on CPU.

(batch, head) units are independent, so `bench.py --gpus N` runs one replica per rank with no exchange
step; what the ranks share is only the timing protocol: barrier, each rank's own time, MAX over ranks,
whole-job value = sum of the ranks' work / slowest rank's time.  This test runs that protocol with
world_size 2 and checks the arithmetic, and that the `--impl reference` arm leaves all work to rank 0.
"""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out_path):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    my_seconds = 0.5 + 0.25 * rank            # rank 1 is the slow one
    my_flops = 3.0e12
    t = torch.tensor([my_seconds], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    value = bench.aggregate([my_flops] * world, float(t.item()))
    # the decision to take another round of steps is taken on the least advanced rank's time, the same everywhere:
    # rank 0 has 1200 ms, rank 1 only 900 ms of a 1 s region -> both go on; at 1200 / 1100 ms both stop
    go_on = bench.more_rounds(1200.0 - 300.0 * rank, 3, 1.0, 100, dist)
    stop = bench.more_rounds(1200.0 - 100.0 * rank, 4, 1.0, 100, dist)
    capped = bench.more_rounds(10.0, 100, 1.0, 100, dist)
    decisions = [None] * world
    dist.all_gather_object(decisions, (go_on, stop, capped))
    if rank == 0:
        with open(out_path, "w") as f:
            json.dump({"value": value, "max_seconds": float(t.item()), "decisions": decisions}, f)
    dist.destroy_process_group()


def test_two_rank_timing_protocol(tmp_path):
    out = str(tmp_path / "agg.json")
    port = 29500 + os.getpid() % 2000
    mp.start_processes(_rank_main, args=(2, port, out), nprocs=2, join=True, start_method="spawn")
    got = json.load(open(out))
    assert got["max_seconds"] == pytest.approx(0.75)
    assert got["value"] == pytest.approx(2 * 3.0 / 0.75)      # TFLOP/s: both ranks' work over the slowest time
    assert got["decisions"] == [[True, False, False], [True, False, False]]


def test_useful_flops_formulas_match_the_papers_counts():
    import bench
    from paper_2012_01114_b200 import inputs
    w = dict(inputs.WORKLOADS["c3"])
    fl = bench.useful_flops(w)
    n, d, B, H, D = 1024, 64, 8, 12, 768
    assert fl["core"] == 2.0 * B * H * 2 * d * n * (n + 1) // 2          # Sec. 5.2: n(n+1)/2 weights, both phases
    assert fl["proj"] == 2.0 * 3 * B * n * D * H * d
    w = dict(inputs.WORKLOADS["c5-n256-symmetric"])
    assert bench.useful_flops(w)["core"] == 2.0 * 256 * 16 * 128 * (256 * 257 // 2 + 256 * 256)   # Sec. 4.1


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "c1"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "c1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0
