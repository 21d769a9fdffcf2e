"""Host-side logic of the N > 1 benchmark path, on CPU with the gloo backend (world size 2).

The hot path has no exchange step: N GPUs run N independent replicas, and the only cross-rank
work is the benchmark's bookkeeping -- the barrier, the maximum of the per-rank times, and the
rule that only rank 0 reports.  These tests run that bookkeeping in two CPU processes."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    dist.barrier()
    mine = 10.0 + 5.0 * rank                              # rank 1 is the slower replica
    slowest = bench.max_over_ranks(mine, dist, torch.device("cpu"))
    line = bench.aggregate_line({"hbm_gbs": 100.0, "value": slowest}, world)
    dist.barrier()
    with open(os.path.join(out_dir, "rank%d.json" % rank), "w") as f:
        json.dump({"slowest": slowest, "line": line}, f)
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregation_with_two_gloo_ranks(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        got = json.load(open(tmp_path / ("rank%d.json" % rank)))
        assert got["slowest"] == 15.0                     # both ranks agree on the slowest replica
        assert got["line"]["n_gpus"] == 2 and got["line"]["hbm_gbs_aggregate"] == 200.0


def test_single_process_needs_no_process_group():
    import bench

    assert bench.max_over_ranks(3.5, None, torch.device("cpu")) == 3.5


def test_reference_arm_reports_from_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
