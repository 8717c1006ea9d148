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


def test_gpus_flag_alone_starts_the_ranks():
    """`python bench.py --gpus 2` with no launcher around it must start two ranks itself.  The launch-check arm goes
    through the same spawner as the GPU arm and reports, over gloo, what the ranks saw."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "launch-check"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["local_ranks_plus_one"] == [1, 2]
    assert lines[0]["max_over_ranks_ms"] == 11.0 and lines[0]["master_addr"] == "127.0.0.1"


def test_clock_sampler_tags_phases_and_survives_a_region_shorter_than_its_period():
    sys.path.insert(0, ROOT)
    import bench
    rows = bench.ClockSampler.parse_rows([
        "2026/01/01 00:00:00.010, 1965, 1965, 300.0, 0x0, Not Active, Not Active, Not Active, Not Active",
        "2026/01/01 00:00:01.000, 1800, 1965, 900.0, 0x4, Not Active, Not Active, Not Active, Active",
        "2026/01/01 00:00:01.020, 1790, 1965, 950.0, 0x4, Not Active, Not Active, Not Active, Active",
        "garbage"])
    assert len(rows) == 3 and rows[1][4] == ["sw_power_cap"]
    import datetime
    t = lambda s: datetime.datetime.strptime(s, "%Y/%m/%d %H:%M:%S.%f").timestamp()
    marks = [(t("2026/01/01 00:00:00.000"), "setup"), (t("2026/01/01 00:00:00.900"), "warmup"),
             (t("2026/01/01 00:00:01.015"), "timed"), (t("2026/01/01 00:00:01.050"), "after")]
    res = bench.ClockSampler.summarise(rows, marks, t("2026/01/01 00:00:02.000"))
    assert res["samples_in_timed_region"] == 1 and res["sm_mhz"] == 1790.0 and res["reasons"] == ["sw_power_cap"]
    # no sample inside the timed region: the samples under load stand in, the set-up phase does not
    marks[2] = (t("2026/01/01 00:00:01.040"), "timed")
    res = bench.ClockSampler.summarise(rows, marks, t("2026/01/01 00:00:02.000"))
    assert res["samples_in_timed_region"] == 0 and res["samples"] == 2 and res["sm_mhz"] == 1795.0
    assert res["phases"]["setup"]["sm_mhz"] == 1965.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
