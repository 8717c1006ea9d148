"""Per-kernel micro-benchmarks of libovggt.so on scaled shapes (CUDA events, warm-up, inputs larger than L2
or an explicit L2 flush between iterations).  One JSON line per kernel.

  python -m paper_2603_05959_b200.microbench all
  python -m paper_2603_05959_b200.microbench attention --M 1374 --N 17758 --heads 16 --iters 20
"""
from __future__ import annotations

import argparse
import json
import os

import torch

from . import binding as B

L2_BYTES = 126 * 1024 * 1024


def _peaks():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    path = os.path.join(root, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return json.load(open(path)), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


class Timer:
    def __init__(self, flush: bool):
        self.flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda") if flush else None

    def run(self, fn, iters: int, warmup: int = 3) -> float:
        """Median milliseconds of fn() over iters launches."""
        for _ in range(warmup):
            fn()
        times = []
        for _ in range(iters):
            if self.flush is not None:
                self.flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b))
        times.sort()
        return times[len(times) // 2]


def _emit(name, ms, shape, bytes_=None, flops=None, extra=None):
    peaks, kind = _peaks()
    rec = {"kernel": name, "shape": shape, "ms": ms, "peaks": kind}
    if bytes_ is not None:
        gbs = bytes_ / (ms * 1e-3) / 1e9
        rec.update({"algorithmic_mb": bytes_ / 1e6, "gb_s": gbs, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"],
                    "frac_of_8tbs_nominal": gbs / 8000.0})
    if flops is not None:
        tf = flops / (ms * 1e-3) / 1e12
        rec.update({"tflops": tf, "frac_of_burst_peak": tf / peaks["bf16_tflops"],
                    "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"]})
    if extra:
        rec.update(extra)
    print(json.dumps(rec), flush=True)
    return rec


def bench_attention(args):
    M, N, H = args.M, args.N, args.heads
    C = H * 64
    g = torch.Generator(device="cuda").manual_seed(1)
    q = torch.randn((M, C), device="cuda", generator=g).bfloat16()
    k = torch.randn((N, C), device="cuda", generator=g).bfloat16()
    v = torch.randn((N, C), device="cuda", generator=g).bfloat16()
    out = torch.empty_like(q)
    scratch = torch.empty(B.lib().ovggt_k_attention_scratch_bytes(M, N, H), dtype=torch.uint8, device="cuda")
    status = torch.zeros(16, dtype=torch.int32, device="cuda")
    if args.tracked_max:
        fn = lambda: B.k_attention(q, k, v, H, out=out, scratch=scratch, status=status)
    else:
        # the library's own call: the key-norm bound exists before the attention runs (the append keeps it)
        kmax2 = B.k_key_norm_bound(k, H)
        sp = torch.cuda.current_stream().cuda_stream
        fn = lambda: B.lib().ovggt_k_attention_bounded(q.data_ptr(), k.data_ptr(), v.data_ptr(), M, N, H, out.data_ptr(),
                                                       scratch.data_ptr(), status.data_ptr(), kmax2.data_ptr(), sp)
    ms = Timer(args.flush).run(fn, args.iters)
    assert int(status[0].item()) == 0
    return _emit("attention (k_attn_tcgen05 + k_attn_merge)", ms, {"M": M, "N": N, "heads": H},
                 flops=4.0 * M * N * C, extra={"kv_mb": 4 * N * C / 1e6,
                                               "softmax_reference": "tracked maximum" if args.tracked_max else "key-norm bound"})


def bench_row_norms(args):
    rows, C = args.rows or (1 << 17), 1024
    x = torch.randn((rows, C), device="cuda").bfloat16()
    ms = Timer(args.flush).run(lambda: B.k_row_norms(x), args.iters)
    return _emit("row_norms (k_row_norms)", ms, {"rows": rows, "C": C}, bytes_=rows * C * 2 + rows * 4)


def bench_diversity(args):
    rows, C = args.rows or (1 << 17), 1024
    x = (torch.randn((rows, C), device="cuda") + 0.25).bfloat16()
    ms = Timer(args.flush).run(lambda: B.k_diversity(x), args.iters)
    return _emit("diversity (k_colsum_partial + k_colsum_final + k_diversity)", ms, {"rows": rows, "C": C},
                 bytes_=2 * rows * C * 2 + rows * 4, extra={"note": "two passes over K by design"})


def bench_select(args):
    N, Bud, batch = args.N or 34142, args.budget or 32768, args.batch
    r = torch.rand((batch, N), device="cuda")
    flags = (torch.rand((batch, N), device="cuda") < 0.05).to(torch.uint8)
    ms = Timer(args.flush).run(lambda: B.k_select(r, flags, Bud), args.iters)
    return _emit("select (k_select)", ms, {"N": N, "budget": Bud, "batch": batch},
                 bytes_=batch * (5 * N + 4 * min(N, Bud)))


def bench_compact(args):
    N, C = args.N or 140000, 1024
    keep = args.budget or (N - 1374 * 8)
    k = torch.randn((N, C), device="cuda").bfloat16()
    v = torch.randn((N, C), device="cuda").bfloat16()
    surv = torch.sort(torch.randperm(N, device="cuda")[:keep]).values.to(torch.int32)
    kd, vd = torch.empty((keep, C), dtype=k.dtype, device="cuda"), torch.empty((keep, C), dtype=k.dtype, device="cuda")
    ms = Timer(args.flush).run(lambda: B.k_compact(k, v, surv, kd, vd), args.iters)
    return _emit("compact (k_compact)", ms, {"rows_in": N, "rows_kept": keep, "C": C}, bytes_=4 * keep * C * 2)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kernel", choices=["attention", "row_norms", "diversity", "select", "compact", "all"])
    ap.add_argument("--M", type=int, default=1374)
    ap.add_argument("--N", type=int, default=0)
    ap.add_argument("--heads", type=int, default=16)
    ap.add_argument("--rows", type=int, default=0)
    ap.add_argument("--budget", type=int, default=0)
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--flush", action="store_true", help="write a 252 MB buffer between iterations")
    ap.add_argument("--tracked-max", action="store_true", help="attention without the key-norm bound")
    args = ap.parse_args()
    torch.cuda.set_device(0)
    todo = ["attention", "row_norms", "diversity", "select", "compact"] if args.kernel == "all" else [args.kernel]
    for name in todo:
        a = argparse.Namespace(**vars(args))
        if name == "attention" and not a.N:
            a.N = 17758
        globals()["bench_" + name](a)


if __name__ == "__main__":
    main()
