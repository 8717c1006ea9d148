"""The multi-GPU benchmark path on CPU: two gloo ranks, replicas only (no data-path collective).  Checks the
max-over-ranks timing, the whole-job rate, the per-rank seeds, and that the reference arm runs on rank 0 alone."""
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_05959_b200 import inputs as gen
from paper_2603_05959_b200 import replicas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each rank "measured" its own times; rank 1 is the slower one on the first, rank 0 on the second
    mine = [10.0 + 5.0 * rank, 7.0 - 2.0 * rank]
    got = replicas.max_over_ranks(mine, world)
    dist.barrier()
    out.put((rank, got, replicas.rank_seed(gen.config_vggt_layer().seed, rank)))
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time_and_add_the_frames():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29517, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1] == [15.0, 7.0]          # element-wise maximum, identical on both ranks
    assert res[0][2] != res[1][2]                          # distinct streams per rank
    assert replicas.aggregate_rate(1000, 15.0, 2) == 2 * 1000 / 15e-3
    assert replicas.max_over_ranks([3.0], 1) == [3.0]      # a single rank needs no process group


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
