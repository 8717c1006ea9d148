#!/usr/bin/env python
"""Benchmark of the OVGGT streaming global-attention step on B200.

A step is one pass of the whole hot path (append, attention, scoring, anchor flags, selection,
compaction) for one frame at one global-attention layer.  Workload: one VGGT-shaped layer, bf16,
1374 tokens/frame, KV budget 16384, 64 anchor tokens - seeded synthetic frames.  The cache is filled
by untimed set-up frames so that every warm-up and timed step runs at steady state (N = B + M rows).

  python bench.py [--gpus N] [--steps K] [--warmup W]          the CUDA library (one JSON line)
  python bench.py --impl reference ...                          the CPU oracle on the host cores

With N > 1 (under torchrun) every rank runs an independent stream of the same shape: replicas only,
no data-path collective; value = frames of all ranks / max-over-ranks time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2603_05959_b200 import inputs as gen  # noqa: E402

METRIC = "frames/sec at fixed KV budget"
UNIT = "frames/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def attention_traffic():
    """DRAM bytes per launch of the attention kernel from its committed ncu summary, or None once the kernel's
    source has changed since that capture."""
    import hashlib
    import re
    prof = os.path.join(ROOT, "profiles", "k_attn_tcgen05_M1374_N17758_H16.md")
    src = os.path.join(ROOT, "paper_2603_05959_b200", "csrc", "attn_tcgen05.cuh")
    try:
        text = open(prof).read()
        sha = re.search(r"^source_sha256: ([0-9a-f]{64})", text, re.M).group(1)
        val = int(re.search(r"^dram_bytes_per_launch: (\d+)", text, re.M).group(1))
        if hashlib.sha256(open(src, "rb").read()).hexdigest() != sha:
            return None
        return val
    except Exception:
        return None


def workload_config(seed_offset: int = 0) -> gen.StreamConfig:
    cfg = gen.config_vggt_layer()
    return cfg.replace(seed=cfg.seed + seed_offset)


def workload_description(cfg: gen.StreamConfig, extra: dict) -> dict:
    d = {"workload": "configs[1]: one VGGT-shaped global-attention layer, bf16, dim 1024 = 16 heads x 64, "
                     "1374 tokens/frame (37x37 patches + 5), KV budget 16384, 64 anchor tokens x K_max 3",
         "tokens_per_frame": cfg.tokens_per_frame, "budget": cfg.budget, "kv_rows_attended": cfg.max_rows,
         "score_mode": "hybrid (Eq. 7)", "state": "steady (cache pre-filled by untimed frames)",
         "l2": "inputs larger than L2: 145 MB of ping-pong K/V buffers plus 11 MB of new tensors per frame, "
               "every frame distinct; no explicit flush"}
    d.update(extra)
    return d


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """nvidia-smi samples of SM clock and throttle reasons while the timed region runs (read-only)."""

    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.uuid = uuid
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.uuid}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def mark_begin(self):
        self.t_begin = time.time()

    def mark_end(self):
        self.t_end = time.time()

    def stop(self) -> dict:
        import datetime
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        try:
            self.proc.terminate()
            self.proc.wait(timeout=5)
        except Exception:
            pass
        try:
            self.out.close()
            rows = [l.strip().split(", ") for l in open(self.path) if l.strip()]
            os.unlink(self.path)
        except Exception:
            return res
        clocks, reasons, mx, power = [], set(), None, []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = []
        for r in rows:
            if len(r) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(r[0].strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
                inside.append(getattr(self, "t_begin", 0) - 0.05 <= ts <= getattr(self, "t_end", 1e18) + 0.05)
            except ValueError:
                inside.append(True)
        if any(inside):
            rows = [r for r, ok in zip([r for r in rows if len(r) >= 9], inside) if ok]
        for r in rows:
            if len(r) < 9:
                continue
            r = r[1:]
            try:
                clocks.append(float(r[0])); mx = float(r[1]); power.append(float(r[2]))
            except ValueError:
                continue
            for name, val in zip(names, r[4:8]):
                if val.strip().lower() == "active":
                    reasons.add(name)
        if clocks:
            top = sorted(clocks)[len(clocks) // 2:]          # samples under load are the upper half at worst
            res.update({"sm_mhz": float(np.median(clocks)), "sm_mhz_upper_half_median": float(np.median(top)),
                        "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(clocks),
                        "power_w_max": max(power) if power else None})
        return res


# ----------------------------------------------------------------------------- CPU oracle leg

class OracleRunner:
    """The CPU oracle as it stands, at steady state: the cache is filled with append + compress only (untimed);
    each timed frame runs the selection path in full and dense attention on `attn_rows` sampled query rows x all
    heads, whose time is scaled to the M rows of a frame."""

    def __init__(self, cfg: gen.StreamConfig, attn_rows: int, threads: int):
        from oracle import oracle as orc
        orc.set_threads(threads)
        self.cfg, self.threads = cfg, threads
        self.layer = orc.OracleLayer.from_stream(cfg)
        self.M = cfg.tokens_per_frame
        self.t = 0
        while self.layer.n_rows < cfg.budget:
            fi = gen.frame_inputs(cfg, self.t)
            self.layer.attend(self.t, fi.q, fi.k, fi.v, compute=False)
            self.layer.compress(fi.resid, fi.conf, fi.rho)
            self.t += 1
        self.rows = np.sort(np.random.default_rng(cfg.seed).choice(self.M, min(attn_rows, self.M),
                                                                    replace=False)).astype(np.int32)
        self.measured = 0.0

    def frame(self) -> float:
        """One frame; returns its extrapolated seconds."""
        fi = gen.frame_inputs(self.cfg, self.t)
        a = time.perf_counter()
        self.layer.attend(self.t, fi.q, fi.k, fi.v, rows=self.rows)
        b = time.perf_counter()
        self.layer.compress(fi.resid, fi.conf, fi.rho)
        c = time.perf_counter()
        self.t += 1
        self.measured += c - a
        return (b - a) * (self.M / len(self.rows)) + (c - b)

    def sample(self, frames: int) -> str:
        return (f"{frames} steady-state frames; selection path in full, dense attention on {len(self.rows)} of "
                f"{self.M} query rows x all heads, attention time scaled by {self.M}/{len(self.rows)} (extrapolated)")


def oracle_rate(cfg: gen.StreamConfig, frames: int, attn_rows: int, threads: int) -> dict:
    run = OracleRunner(cfg, attn_rows, threads)
    per_frame = float(np.mean([run.frame() for _ in range(frames)]))
    return {"value": 1.0 / per_frame, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": run.sample(frames),
            "measured_seconds": run.measured, "ms_per_frame_extrapolated": per_frame * 1e3}


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = workload_config()
    threads = host_cores()
    # one bounded sample (a frame with attention on sampled rows) per step; the whole run is bounded in time
    run = OracleRunner(cfg, args.ref_rows, threads)
    per = []
    t0 = time.perf_counter()
    for i in range(args.warmup + args.steps):
        sec = run.frame()
        if i >= args.warmup:
            per.append(sec * 1e3)
        if time.perf_counter() - t0 > 120 and i >= args.warmup:
            break
    res = {"sample": run.sample(len(per)) + ("; stopped after 120 s" if len(per) < args.steps else "")}
    ms = float(np.mean(per))
    value = 1e3 / ms
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(per), "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_description(cfg, {"reference": "CPU oracle (oracle/), host cores only"}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": res["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- the CUDA library

def run_ours(args) -> None:
    import torch
    import torch.distributed as dist
    from paper_2603_05959_b200 import binding as B
    from paper_2603_05959_b200 import replicas
    from paper_2603_05959_b200.stream import DeviceFrame

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    cfg = workload_config(seed_offset=replicas.rank_seed(0, rank))
    M, C, Bud = cfg.tokens_per_frame, cfg.dim, cfg.budget
    K, W = args.steps, args.warmup
    fill = -(-Bud // M) + 1                           # frames until the cache is full, plus one
    n_e2e = min(K, args.e2e_steps)
    n_prof = min(K, args.profile_steps)
    need = fill + W + K + n_prof + n_e2e
    pool = min(need, args.pool)
    host_frames = [gen.frame_inputs(cfg, t) for t in range(pool)]
    frames = [DeviceFrame(cfg, fi, dev) for fi in host_frames]
    pinned = [DeviceFrame(cfg, fi, None, pin=True) for fi in host_frames[:min(pool, 8)]]
    cache = B.OvggtCache.from_stream(cfg, device=dev)
    out = cache.new_out()
    stream = torch.cuda.current_stream()
    t_id = 0

    def step(t):
        f = frames[t % pool]
        cache.layer_step(0, t, f.q, f.k, f.v, f.resid, f.conf, f.rho, out=out, stream=stream)

    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    sampler.start()
    for _ in range(fill):
        step(t_id); t_id += 1
    for _ in range(W):
        step(t_id); t_id += 1
    torch.cuda.synchronize()
    assert cache.stats(0)["n_cached"] == Bud

    # ---- timed region: K steps, device-resident inputs, CUDA events on the launching stream
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.mark_begin()
    launches0 = B.kernel_launches()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    ev[0].record(stream)
    for i in range(K):
        step(t_id); t_id += 1
        ev[i + 1].record(stream)
    torch.cuda.synchronize()
    sampler.mark_end()
    if world > 1:
        dist.barrier()
    launches = B.kernel_launches() - launches0
    total_ms = ev[0].elapsed_time(ev[K])
    per_step = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(K)])

    # ---- per-kernel device time (events around each kernel class; separate pass, same stream of frames)
    cache.set_overlap(False)           # one kernel class at a time: the two halves of a step on one stream
    cache.profile_enable(True)
    for _ in range(n_prof):
        step(t_id); t_id += 1
    prof = cache.profile_read(reset=True)
    cache.profile_enable(False)
    cache.set_overlap(True)
    clocks = sampler.stop()

    # ---- end to end: host buffers through the C ABI, copies inside the timed region
    out_host = [torch.empty((M, C), dtype=out.dtype).pin_memory() for _ in range(2)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for i in range(n_e2e):
        f = pinned[i % len(pinned)]
        cache.layer_step_host(0, t_id, f.q, f.k, f.v, f.resid, f.conf, f.rho, out_host[i % 2], stream=stream)
        t_id += 1
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    st = cache.stats(0)
    assert st["device_status"] == 0 and st["n_cached"] == Bud

    # ---- max over ranks
    total_ms, e2e_ms = replicas.max_over_ranks([total_ms, e2e_ms], world, dev)
    value = replicas.aggregate_rate(K, total_ms, world)
    e2e_value = replicas.aggregate_rate(n_e2e, e2e_ms, world)

    if rank == 0:
        peaks, peak_kind = load_peaks()
        N = Bud + M
        attn_flops = 4.0 * M * N * C
        attn_ms = prof["attention"]["ms"] / max(1, prof["attention"]["count"])
        achieved = attn_flops / (attn_ms * 1e-3) / 1e12 if attn_ms > 0 else 0.0
        peak = float(peaks["bf16_tflops"])
        eb = cfg.elem_bytes
        kernels = {}
        alg_bytes = {"append": 4 * M * C * eb, "row_norms": M * C * eb + 4 * M,
                     "diversity": Bud * C * eb + 4 * Bud + M * C * eb + 4 * M, "select": 4 * N + N + 4 * Bud,
                     "compact": 4 * Bud * C * eb}
        for name, rec in prof.items():
            ms = rec["ms"] / max(1, rec["count"])
            kernels[name] = {"ms": ms}
            if name in alg_bytes and ms > 0:
                gbs = alg_bytes[name] / (ms * 1e-3) / 1e9
                kernels[name].update({"algorithmic_mb": alg_bytes[name] / 1e6, "gb_s": gbs,
                                      "frac_of_measured_hbm": gbs / float(peaks["hbm_gbs"]),
                                      "frac_of_8tbs_nominal": gbs / 8000.0})
        kernels["attention"].update({"tflops": achieved, "frac_of_burst_peak": achieved / peak,
                                     "frac_of_sustained_peak": achieved / float(peaks["bf16_tflops_sustained"])})
        half = per_step[len(per_step) // 2:]
        slope = float(np.polyfit(np.arange(K), per_step, 1)[0]) if K >= 3 else 0.0
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": workload_description(cfg, {"parallelism": "replicas only" if world > 1 else "single GPU",
                                                 "setup_frames": fill, "input_pool_frames": pool}),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 4 * M * C * eb + 4 * cfg.n_patches,
                    "d2h_bytes_per_step": M * C * eb, "steps": n_e2e, "ms_per_step": e2e_ms / max(1, n_e2e)},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": {"kernel": "k_attn_tcgen05 (+ k_attn_merge)", "bound": "tensor", "achieved": achieved,
                         "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                         "peak_kind": f"{peak_kind} burst cuBLAS bf16 peak", "traffic": None,
                         "algorithmic_flops": attn_flops, "launch_ms": attn_ms},
            "kernels": kernels,
            "ms_per_frame": {"median": float(np.median(per_step)), "max": float(per_step.max()),
                             "min": float(per_step.min()), "slope_ms_per_frame": slope,
                             "max_over_median": float(per_step.max() / np.median(per_step)),
                             "second_half_median": float(np.median(half))},
        }
        line["roofline"]["traffic"] = attention_traffic()
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = oracle_rate(cfg, frames=args.cpu_frames, attn_rows=args.ref_rows,
                                               threads=host_cores())
        else:
            line["cpu_baseline"] = None
        print(json.dumps(line))
    cache.destroy()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--pool", type=int, default=160, help="distinct frames kept on the device (cycled beyond)")
    ap.add_argument("--e2e-steps", type=int, default=200)
    ap.add_argument("--profile-steps", type=int, default=100)
    ap.add_argument("--cpu-frames", type=int, default=8)
    ap.add_argument("--ref-rows", type=int, default=96)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
