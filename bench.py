#!/usr/bin/env python
"""Benchmark of the OVGGT streaming global-attention step on B200.

A step is one pass of the whole hot path (append, attention, scoring, anchor flags, selection,
compaction) for one frame at one global-attention layer.  Default workload (c2): one VGGT-shaped layer, bf16,
1374 tokens/frame, KV budget 16384, 64 anchor tokens - seeded synthetic frames.  The cache is filled
by untimed set-up frames so that every warm-up and timed step runs at steady state (N = B + M rows).

  python bench.py [--gpus N] [--steps K] [--warmup W]          the CUDA library on c2 (one JSON line)
  python bench.py --config {c1,c2,c3,c4,c5} ...                 the other workload shapes (one JSON line each)
  python bench.py --impl reference ...                          the CPU oracle on the host cores

With N > 1 every rank runs independent streams of the same shape: replicas only, no data-path collective;
value = frames of all ranks / max-over-ranks time.  Started without torchrun, `--gpus N` launches the N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
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
L2_MB = 126


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


WORKLOADS = {
    "c1": "configs[0]: tiny single global-attention layer, fp32, dim 256 = 4 heads x 64, 69 tokens/frame (8x8 patches "
          "+ 5), 16-frame stream, KV budget 256, 8 anchor tokens",
    "c2": "configs[1]: one VGGT-shaped global-attention layer, bf16, dim 1024 = 16 heads x 64, "
          "1374 tokens/frame (37x37 patches + 5), KV budget 16384, 64 anchor tokens x K_max 3",
    "c3": "configs[2]: stack of 24 global-attention layers, bf16, dim 1024, each with its own KV cache of 8192 tokens, "
          "random-init QKV/out projections N(0, 0.02), 1374 tokens/frame, 64 anchor tokens per layer",
    "c4": "configs[3]: alternating aggregator, bf16, 24 frame-attention + 24 global-attention blocks, dim 1024, 16 "
          "heads, MLP 4096, random-init N(0, 0.02), 1041 tokens/frame (37x28 patches + 5), per-layer budget 12288, "
          "64 anchor tokens",
    "c5": "configs[4]: ultra-long stream, one VGGT-shaped layer bf16, 1374 tokens/frame, budgets {4096, 16384, 32768} "
          "x anchor tokens {0, 64, 256} x both score modes, residual gain drifting +0.1 (log-mean) per 1000 frames",
}


def stream_config(name: str, seed_offset: int = 0) -> gen.StreamConfig:
    cfg = {"c1": gen.config_tiny, "c2": gen.config_vggt_layer, "c3": gen.config_stack24,
           "c4": gen.config_aggregator, "c5": gen.config_ultra_long}[name]()
    return cfg.replace(seed=cfg.seed + seed_offset)


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """nvidia-smi samples of SM clock and throttle reasons (read-only), taken every 20 ms from before the set-up
    frames until after the timed region; samples are tagged by the phase they fall into."""

    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, uuid: str):
        self.uuid = uuid
        self.proc = None
        self.path = None
        self.marks = []          # (wall time, phase that starts here)

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.uuid}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        self.mark("setup")

    def mark(self, phase: str):
        self.marks.append((time.time(), phase))

    @staticmethod
    def parse_rows(lines):
        """[(timestamp or None, sm, max_sm, power, [active reason names])] from nvidia-smi csv lines."""
        import datetime
        out = []
        for l in lines:
            r = [x.strip() for x in l.strip().split(",")]
            if len(r) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(r[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
            except ValueError:
                ts = None
            try:
                sm, mx, pw = float(r[1]), float(r[2]), float(r[3])
            except ValueError:
                continue
            out.append((ts, sm, mx, pw, [n for n, v in zip(ClockSampler.NAMES, r[5:9]) if v.lower() == "active"]))
        return out

    @staticmethod
    def summarise(rows, marks, t_end):
        """Per-phase medians; the headline figures are the timed phase's when it has samples, else those of all
        samples under load (so a region shorter than the sampling period still gets a clock record)."""
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "phases": {}}
        if not rows:
            return res
        bounds = [(t, p) for t, p in marks] + [(t_end, None)]
        tagged = {}
        for ts, sm, mx, pw, why in rows:
            phase = "untagged"
            if ts is not None:
                for (t0, p), (t1, _) in zip(bounds, bounds[1:]):
                    if t0 - 0.01 <= ts <= t1 + 0.01:
                        phase = p
            tagged.setdefault(phase, []).append((sm, mx, pw, why))
        for p, rs in tagged.items():
            res["phases"][p] = {"samples": len(rs), "sm_mhz": float(np.median([r[0] for r in rs])),
                                "power_w_max": max(r[2] for r in rs),
                                "reasons": sorted({n for r in rs for n in r[3]})}
        use = tagged.get("timed") or [r for p, rs in tagged.items() if p != "setup" for r in rs] or \
            [r for rs in tagged.values() for r in rs]
        res.update({"sm_mhz": float(np.median([r[0] for r in use])), "sm_max_mhz": use[0][1],
                    "reasons": sorted({n for r in use for n in r[3]}), "samples": len(use),
                    "samples_in_timed_region": len(tagged.get("timed", [])),
                    "power_w_max": max(r[2] for r in use)})
        return res

    def stop(self) -> dict:
        t_end = time.time()
        if self.proc is None:
            return self.summarise([], self.marks, t_end)
        try:
            self.proc.terminate()
            self.proc.wait(timeout=5)
        except Exception:
            pass
        try:
            self.out.close()
            lines = open(self.path).read().splitlines()
            os.unlink(self.path)
        except Exception:
            lines = []
        return self.summarise(self.parse_rows(lines), self.marks, t_end)


# ----------------------------------------------------------------------------- CPU oracle leg

class OracleRunner:
    """The CPU oracle as it stands, at steady state: the cache is filled with append + compress only (untimed);
    each timed frame runs the selection path in full and dense attention on `attn_rows` sampled query rows x all
    heads, whose time is scaled to the M rows of a frame."""

    def __init__(self, cfg: gen.StreamConfig, attn_rows: int, threads: int):
        from oracle import oracle as orc
        self.orc = orc
        orc.set_threads(host_cores())                 # the untimed fill uses every core
        self.cfg, self.threads = cfg, threads
        self.layer = orc.OracleLayer.from_stream(cfg)
        self.M = cfg.tokens_per_frame
        self.t = 0
        while self.layer.n_rows < cfg.budget and self.t < cfg.n_frames + 64:
            fi = gen.frame_inputs(cfg, self.t)
            self.layer.attend(self.t, fi.q, fi.k, fi.v, compute=False)
            self.layer.compress(fi.resid, fi.conf, fi.rho)
            self.t += 1
        self.rows = np.sort(np.random.default_rng(cfg.seed).choice(self.M, min(attn_rows, self.M),
                                                                    replace=False)).astype(np.int32)
        self.measured = 0.0

    def frame(self, threads=None) -> float:
        """One frame; returns its extrapolated seconds."""
        self.orc.set_threads(threads or self.threads)
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
        full = len(self.rows) == self.M
        att = "dense attention in full" if full else (
            f"dense attention on {len(self.rows)} of {self.M} query rows x all heads, attention time scaled by "
            f"{self.M}/{len(self.rows)} (extrapolated)")
        return f"{frames} steady-state frames; selection path in full, {att}"


def oracle_rate(cfg: gen.StreamConfig, frames: int, attn_rows: int, threads: int, single_rows: int = 0) -> dict:
    """All-cores rate over `frames` frames and, with single_rows > 0, a single-thread rate on one frame with fewer
    sampled attention rows (the oracle is the same; only its OpenMP thread count differs)."""
    run = OracleRunner(cfg, attn_rows, threads)
    per_frame = float(np.mean([run.frame() for _ in range(frames)]))
    res = {"value": 1.0 / per_frame, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": run.sample(frames),
           "measured_seconds": run.measured, "ms_per_frame_extrapolated": per_frame * 1e3}
    if single_rows > 0:
        one = OracleRunner.__new__(OracleRunner)
        one.__dict__.update(run.__dict__)
        one.rows = run.rows[:: max(1, len(run.rows) // single_rows)][:single_rows]
        one.measured = 0.0
        sec = one.frame(threads=1)
        res["single_thread"] = {"value": 1.0 / sec, "unit": UNIT, "cores": 1, "sample": one.sample(1),
                                "measured_seconds": one.measured, "ms_per_frame_extrapolated": sec * 1e3}
    return res


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = stream_config(args.config)
    if args.config == "c5":
        cfg = gen.config_ultra_long()
    cfg = cfg.replace(n_layers=1)
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
            "config": workload_description(args.config, cfg, {"reference": "CPU oracle (oracle/), host cores only; one "
                                                              "layer-step per step"}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": res["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_description(name: str, cfg: gen.StreamConfig, extra: dict) -> dict:
    d = {"workload": WORKLOADS[name], "tokens_per_frame": cfg.tokens_per_frame, "budget": cfg.budget,
         "kv_rows_attended": cfg.max_rows, "score_mode": "hybrid (Eq. 7)",
         "state": "steady (cache pre-filled by untimed frames)"}
    d.update(extra)
    return d


# ----------------------------------------------------------------------------- the CUDA library

def init_rank():
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    return world, rank, dev


def kernel_table(prof: dict, alg_bytes: dict, peaks: dict, sm_mhz) -> dict:
    """Per-class device time of the profiling pass (CUDA events around each class, one class at a time), in
    microseconds and in SM cycles at the sampled clock, with the algorithmic bytes against both HBM figures."""
    kernels = {}
    for name, rec in prof.items():
        ms = rec["ms"] / max(1, rec["count"])
        kernels[name] = {"ms": ms, "launch_groups": rec["count"]}
        if sm_mhz:
            kernels[name]["sm_cycles"] = ms * 1e-3 * sm_mhz * 1e6
        if name in alg_bytes and ms > 0:
            gbs = alg_bytes[name] / (ms * 1e-3) / 1e9
            kernels[name].update({"algorithmic_mb": alg_bytes[name] / 1e6, "gb_s": gbs,
                                  "frac_of_measured_hbm": gbs / float(peaks["hbm_gbs"]),
                                  "frac_of_8tbs_nominal": gbs / 8000.0})
    return kernels


def run_c2(args) -> None:
    """The headline workload (and c1 with --config c1): single-layer streams at steady state."""
    import torch
    import torch.distributed as dist
    from paper_2603_05959_b200 import binding as B
    from paper_2603_05959_b200 import replicas
    from paper_2603_05959_b200.harness import RotatingLayers, flatness, time_per_step
    from paper_2603_05959_b200.stream import DeviceFrame

    world, rank, dev = init_rank()
    cfg = stream_config(args.config, seed_offset=replicas.rank_seed(0, rank))
    M, C, Bud = cfg.tokens_per_frame, cfg.dim, cfg.budget
    K, W = args.steps, args.warmup
    compaction = B.COMPACT_STABLE_GATHER if args.compaction == "stable" else B.COMPACT_FILL_HOLES
    kv_mb = 2 * cfg.max_rows * C * cfg.elem_bytes / 1e6 * (2 if compaction == B.COMPACT_STABLE_GATHER else 1)
    # A step re-reads its stream's K/V cache.  One cache (73 MB at c2) would stay in the 126 MB L2 from one step to
    # the next, which no 24-layer model would see; so the steps go round several independent streams.
    R = args.streams if args.streams > 0 else max(1, int(np.ceil(2.2 * L2_MB / kv_mb)))
    if args.config == "c1" and args.streams <= 0:
        R = 1                        # the tiny fp32 case: nothing about it is larger than L2
    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    sampler.start()
    pool = args.pool
    rot = RotatingLayers(cfg, R, dev, pool, compaction=compaction)
    pinned = [DeviceFrame(cfg, fi, None, pin=True) for fi in rot.host_frames[:min(pool, 8)]]
    stream = torch.cuda.current_stream()
    n_e2e = min(K, args.e2e_steps)
    n_prof = min(K, args.profile_steps)
    for _ in range(rot.fill_frames()):
        rot.step(stream)
    sampler.mark("warmup")
    for _ in range(W):
        rot.step(stream)
    torch.cuda.synchronize()
    rot.check()

    # ---- timed region: K steps, device-resident inputs, CUDA events on the launching stream
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.mark("timed")
    launches0 = B.kernel_launches()
    total_ms, per_step = time_per_step(lambda: rot.step(stream), K, stream)
    sampler.mark("after")
    if world > 1:
        dist.barrier()
    launches = B.kernel_launches() - launches0

    # ---- per-kernel device time (events around each kernel class; separate pass, same streams of frames)
    rot.set_overlap(False)           # one kernel class at a time: the two halves of a step on one stream
    rot.profile_enable(True)
    for _ in range(n_prof):
        rot.step(stream)
    prof = rot.profile_read()
    rot.profile_enable(False)
    rot.set_overlap(True)

    # ---- one stream alone, its cache L2-resident between steps (reported beside the headline, not as it)
    single_ms = None
    if R > 1 and rank == 0:
        one = RotatingLayers(cfg, 1, dev, min(pool, 32), compaction=compaction)
        for _ in range(one.fill_frames() + W):
            one.step(stream)
        torch.cuda.synchronize()
        ks = min(K, 500)
        single_ms = time_per_step(lambda: one.step(stream), ks, stream)[0] / ks
        one.destroy()

    # ---- end to end: host buffers through the C ABI, copies inside the timed region
    out_host = [torch.empty((M, C), dtype=rot.out.dtype).pin_memory() for _ in range(2)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    sampler.mark("e2e")
    e0.record(stream)
    for i in range(n_e2e):
        rot.step_host(pinned, out_host, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    rot.check()
    clocks = sampler.stop()

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
        fill = compaction == B.COMPACT_FILL_HOLES
        # hole filling: the append launch also carries the previous step's moves (at most M rows of K and V read and
        # written again); stable gather: all B rows are read and written by the compaction
        alg_bytes = {"append": (8 if fill else 4) * M * C * eb, "row_norms": M * C * eb + 4 * M,
                     "diversity": Bud * C * eb + 4 * Bud + M * C * eb + 4 * M, "select": 4 * N + N + 4 * Bud,
                     "compact": 4 * Bud * C * eb}
        kernels = kernel_table(prof, alg_bytes, peaks, clocks.get("sm_mhz"))
        if cfg.dtype == gen.DTYPE_BF16:
            kernels["attention"].update({"tflops": achieved, "frac_of_burst_peak": achieved / peak,
                                         "frac_of_sustained_peak": achieved / float(peaks["bf16_tflops_sustained"])})
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if cfg.dtype == gen.DTYPE_BF16 else "f32", "data": "synthetic",
            "config": workload_description(args.config, cfg, {
                "parallelism": "replicas only" if world > 1 else "single GPU",
                "compaction": "hole filling (one K/V buffer)" if fill else "stable gather (two K/V buffers)",
                "streams_in_rotation": R, "setup_frames": rot.fill_frames(), "input_pool_frames": pool,
                "l2": (f"inputs larger than L2: {R} independent streams of this configuration take turns, so a step "
                       f"finds neither its {kv_mb:.0f} MB K/V cache ({R * kv_mb:.0f} MB in all) nor its new "
                       f"tensors in the {L2_MB} MB L2; no explicit flush") if R * kv_mb > 1.5 * L2_MB else
                      "working set smaller than L2 (a parity-sized case, not a bandwidth measurement)"}),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 4 * M * C * eb + 4 * cfg.n_patches,
                    "d2h_bytes_per_step": M * C * eb, "steps": n_e2e, "ms_per_step": e2e_ms / max(1, n_e2e)},
            "gpu_launches": int(launches),
            "launches_per_step": launches / K,
            "clocks": clocks,
            "roofline": {"kernel": "k_attn_tcgen05", "bound": "tensor", "achieved": achieved,
                         "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                         "peak_kind": f"{peak_kind} burst cuBLAS bf16 peak", "traffic": attention_traffic(),
                         "algorithmic_flops": attn_flops, "launch_ms": attn_ms,
                         # the launch is timed right after the K timed steps, at the clocks the step itself ran at;
                         # the same figure against the sustained (power-capped) cuBLAS peak, for long runs
                         "frac_of_sustained_peak": achieved / float(peaks["bf16_tflops_sustained"])},
            "kernels": kernels,
            "ms_per_frame": flatness(per_step),
            "single_stream_l2_resident": None if single_ms is None else
            {"ms_per_step": single_ms, "value": 1e3 / single_ms, "note": "one stream alone: its K/V cache stays in L2 "
             "between steps; context only"},
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = oracle_rate(cfg, frames=args.cpu_frames, attn_rows=args.ref_rows,
                                               threads=host_cores(), single_rows=8)
        else:
            line["cpu_baseline"] = None
        print(json.dumps(line))
    rot.destroy()
    if world > 1:
        dist.destroy_process_group()


def run_stack(args) -> None:
    """c3 (projection stack) and c4 (alternating aggregator): a step is one frame through all 24 layers; the
    library's share of the device time is measured by events around its calls, the scaffold's is the rest."""
    import torch
    from paper_2603_05959_b200 import binding as B
    from paper_2603_05959_b200 import harness as H

    world, rank, dev = init_rank()
    if world > 1:
        raise SystemExit("--config c3 / c4 run on one GPU")
    cfg = stream_config(args.config)
    M, C, Bud, L = cfg.tokens_per_frame, cfg.dim, cfg.budget, cfg.n_layers
    K = min(args.steps, 200)
    W = args.warmup
    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    sampler.start()
    model = H.ProjectionStack(cfg, dev, matmul=args.scaffold) if args.config == "c3" else \
        H.Aggregator(cfg, dev, matmul=args.scaffold, frame_attention=args.scaffold)
    stream = torch.cuda.current_stream()
    fill = -(-Bud // M) + 1
    pool = min(args.pool, 24)
    side = [H.frame_side_inputs(cfg, t, dev, L if args.config == "c3" else 0) for t in range(pool)]
    emb = [H.patch_embeddings(cfg, t, dev) for t in range(pool)]
    t_id = 0

    def frame(lib=None):
        nonlocal t_id
        conf, rho, resid = side[t_id % pool]
        if args.config == "c3":
            model.frame(t_id, emb[t_id % pool], resid, conf, rho, stream, lib)
        else:
            model.frame(t_id, emb[t_id % pool], conf, rho, stream, lib)
        t_id += 1

    for _ in range(fill):
        frame()
    sampler.mark("warmup")
    for _ in range(W):
        frame()
    torch.cuda.synchronize()
    sampler.mark("timed")
    launches0 = B.kernel_launches()
    total_ms, per_frame = H.time_per_step(frame, K, stream)
    launches = B.kernel_launches() - launches0
    sampler.mark("split")
    # library / scaffold split: a second pass with events around every library call
    lib = H._Timer(stream)
    n_split = min(K, 20)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(n_split):
        frame(lib)
    b.record(stream)
    lib_ms = lib.total_ms() / n_split
    all_ms = a.elapsed_time(b) / n_split
    # the library's own per-class times
    model.cache.set_overlap(False)
    model.cache.profile_enable(True)
    for _ in range(min(K, 10)):
        frame()
    prof = model.cache.profile_read(reset=True)
    model.cache.profile_enable(False)
    model.cache.set_overlap(True)
    for l in range(L):
        st = model.cache.stats(l)
        assert st["device_status"] == 0 and st["n_cached"] == Bud, (l, st)
    clocks = sampler.stop()
    peaks, peak_kind = load_peaks()
    N = Bud + M
    attn_flops = 4.0 * M * N * C
    attn_ms = prof["attention"]["ms"] / max(1, prof["attention"]["count"])
    achieved = attn_flops / (attn_ms * 1e-3) / 1e12
    peak = float(peaks["bf16_tflops"])
    eb = cfg.elem_bytes
    alg_bytes = {"append": 8 * M * C * eb, "row_norms": M * C * eb + 4 * M,
                 "diversity": Bud * C * eb + 4 * Bud + M * C * eb + 4 * M, "select": 4 * N + N + 4 * Bud}
    # c4 compresses all layers with one call at the end of the frame: its diversity and select launches are the batched
    # ones (one launch group per frame covering L layers), so their algorithmic bytes are L layers' worth
    n_frames_prof = min(K, 10)
    for name in ("diversity", "select"):
        if prof[name]["count"] == n_frames_prof:
            alg_bytes[name] *= L
    kernels = kernel_table(prof, alg_bytes, peaks, clocks.get("sm_mhz"))
    for name in ("diversity", "select"):
        kernels[name]["layers_per_launch_group"] = L if prof[name]["count"] == n_frames_prof else 1
    line = {"metric": METRIC, "value": K / (total_ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": workload_description(args.config, cfg, {
                "step": f"one frame through all {L} layers (scaffold in torch + library)",
                "l2": f"inputs larger than L2: {L} layer caches of {2 * cfg.max_rows * C * eb / 1e6:.0f} MB each are "
                      "visited in turn; no explicit flush"}),
            "time_split_ms_per_frame": {"all": all_ms, "library": lib_ms, "scaffold": all_ms - lib_ms,
                                        "library_layer_steps_per_s": L / (lib_ms * 1e-3),
                                        "note": "events around every call of the streaming step's entry points in a "
                                                f"separate pass of {n_split} frames; scaffold = projections, MLPs, "
                                                "LayerNorm, frame attention with random-init weights "
                                                f"(matmuls and frame attention on: {args.scaffold})"},
            "e2e": None, "gpu_launches": int(launches), "launches_per_step": launches / K, "clocks": clocks,
            "roofline": {"kernel": "k_attn_tcgen05", "bound": "tensor", "achieved": achieved, "peak": peak,
                         "unit": "TFLOP/s", "frac": achieved / peak, "peak_kind": f"{peak_kind} burst cuBLAS bf16 peak",
                         "traffic": None, "algorithmic_flops": attn_flops, "launch_ms": attn_ms},
            "kernels": kernels,
            "ms_per_frame": H.flatness(per_frame)}
    if not args.no_cpu_baseline:
        # the oracle's share is one layer-step of this shape; a frame is L of them
        one = oracle_rate(cfg.replace(n_layers=1), frames=max(1, args.cpu_frames // 4), attn_rows=min(args.ref_rows, 48),
                          threads=host_cores())
        one["value"] /= L
        one["sample"] += f"; one layer-step timed, a frame taken as {L} of them"
        line["cpu_baseline"] = one
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line))
    model.destroy()


def run_sweep(args) -> None:
    """c5: budget x anchor tokens x score mode, 10,000 frames each (or --steps), one stream per point."""
    import torch
    from paper_2603_05959_b200 import binding as B
    from paper_2603_05959_b200 import harness as H
    from paper_2603_05959_b200.stream import DeviceFrame

    world, rank, dev = init_rank()
    if world > 1:
        raise SystemExit("--config c5 runs on one GPU")
    T = args.steps
    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    sampler.start()
    sampler.mark("timed")
    stream = torch.cuda.current_stream()
    peaks, peak_kind = load_peaks()
    points = []
    launches0 = B.kernel_launches()
    base = gen.config_ultra_long()
    blocks = max(1, -(-T // 1000))
    # 12 distinct frames per block of 1000, drawn at that block's gain level (shared by every point of the sweep)
    frames = {blk: [DeviceFrame(base, gen.frame_inputs(base, blk * 1000 + i), dev) for i in range(12)]
              for blk in range(blocks)}
    for budget in (4096, 16384, 32768):
        for anchors in (0, 64, 256):
            for mode in (gen.SCORE_HYBRID, gen.SCORE_RESIDUAL_STORED):
                cfg = gen.config_ultra_long(budget, anchors, mode)
                cache = B.OvggtCache.from_stream(cfg, device=dev)
                out = cache.new_out()
                t_id = 0

                def step():
                    nonlocal t_id
                    f = frames[min(blocks - 1, t_id // 1000)][t_id % 12]
                    cache.layer_step(0, t_id, f.q, f.k, f.v, f.resid, f.conf, f.rho, out=out, stream=stream)
                    t_id += 1

                total_ms, per = H.time_per_step(step, T, stream)
                st = cache.stats(0)
                assert st["device_status"] == 0 and st["n_cached"] == min(budget, T * cfg.tokens_per_frame)
                warm = -(-budget // cfg.tokens_per_frame) + 20           # fill phase + 20 frames excluded
                steady = per[min(warm, len(per) - 1):]
                fl = H.flatness(steady)
                N = budget + cfg.tokens_per_frame
                points.append({"budget": budget, "anchor_tokens": anchors,
                               "score_mode": "hybrid" if mode == gen.SCORE_HYBRID else "residual_stored",
                               "frames": T, "frames_per_s_steady": 1e3 / fl["median"], "ms_per_frame": fl,
                               "kv_rows_attended": N, "n_active_anchors": st["n_active_anchors"],
                               "evicted_total": st["evicted_total"],
                               "attention_gflop_per_frame": H.attention_flops(cfg.tokens_per_frame, N, cfg.dim) / 1e9})
                cache.destroy()
                del cache, out
    clocks = sampler.stop()
    mid = next(p for p in points if p["budget"] == 16384 and p["anchor_tokens"] == 64 and p["score_mode"] == "hybrid")
    cfg = gen.config_ultra_long()
    line = {"metric": METRIC, "value": mid["frames_per_s_steady"], "unit": UNIT, "n_gpus": 1, "steps": T,
            "warmup": 0, "ms_per_step": mid["ms_per_frame"]["median"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_description("c5", cfg, {
                "value_is": "steady-state frames/s of the point budget 16384, 64 anchor tokens, hybrid score",
                "l2": "one stream per point, its K/V cache re-read every step (22 to 140 MB: the small budgets are "
                      "L2-resident, which is what a single-layer stream does); 12 distinct input frames per 1000"}),
            "sweep": points, "e2e": None, "gpu_launches": int(B.kernel_launches() - launches0), "clocks": clocks,
            "roofline": None, "cpu_baseline": None}
    print(json.dumps(line))


def run_launch_check(args) -> None:
    """What every rank of a `--gpus N` launch sees, gathered over gloo without touching a GPU: a check of the
    launcher itself (ranks started, environment set, rendezvous on 127.0.0.1)."""
    import torch
    import torch.distributed as dist
    from paper_2603_05959_b200 import replicas
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    seen = torch.zeros(world, dtype=torch.int64)
    seen[rank] = 1 + int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.all_reduce(seen)
    slowest = replicas.max_over_ranks([10.0 + rank], world)[0]
    if rank == 0:
        print(json.dumps({"impl": "launch-check", "n_gpus": world, "local_ranks_plus_one": seen.tolist(),
                          "max_over_ranks_ms": slowest, "master_addr": os.environ.get("MASTER_ADDR")}))
    if world > 1:
        dist.destroy_process_group()


def respawn_under_torchrun(args) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks (one per GPU) and pass the arguments on."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "launch-check"])
    ap.add_argument("--config", default="c2", choices=sorted(WORKLOADS))
    ap.add_argument("--compaction", default="fill", choices=["fill", "stable"])
    ap.add_argument("--scaffold", default="library", choices=["library", "torch"],
                    help="c3 / c4: projections, MLPs and frame attention on the library's tcgen05 kernels or on torch")
    ap.add_argument("--streams", type=int, default=0, help="independent streams in rotation (0: enough to exceed L2)")
    ap.add_argument("--pool", type=int, default=160, help="distinct frames kept on the device (cycled beyond)")
    ap.add_argument("--e2e-steps", type=int, default=200)
    ap.add_argument("--profile-steps", type=int, default=100)
    ap.add_argument("--cpu-frames", type=int, default=8)
    ap.add_argument("--ref-rows", type=int, default=96)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        raise SystemExit(respawn_under_torchrun(args))
    if args.impl == "launch-check":
        run_launch_check(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.config in ("c1", "c2"):
        run_c2(args)
    elif args.config in ("c3", "c4"):
        run_stack(args)
    else:
        run_sweep(args)


if __name__ == "__main__":
    main()
