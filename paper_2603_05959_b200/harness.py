"""Workload harnesses around the library for the benchmark and the GPU tests.

The library is the hot path: cache append, attention over [cache ; frame], scoring, anchor flags, selection and
compaction.  What a model wraps around it (projections, LayerNorm, frame attention, MLP) is *scaffold*: random-init
torch ops that exist here only to give the library inputs with the right shapes and data dependencies.  Scaffold
time is measured separately from library time and never counted as the library's.

  RotatingLayers   several independent streams of one single-layer configuration, visited in turn, so that a step
                   never finds its own K/V cache in L2 from the step before
  ProjectionStack  24 global-attention layers, each with its own cache, with random-init QKV / output projections
  Aggregator       alternating frame-attention and global-attention blocks with MLPs; the global block runs
                   attend -> MLP -> compress with the block's real MLP residual as the activation score's input
"""
from __future__ import annotations

from typing import Callable, List, Optional

import numpy as np
import torch

from . import binding as B
from . import inputs as gen
from .stream import DeviceFrame


class RotatingLayers:
    """R independent handles of one single-layer configuration; step i goes to handle i % R."""

    def __init__(self, cfg: gen.StreamConfig, n_streams: int, device, pool_frames: int, seed_offset: int = 0,
                 compaction: int = B.COMPACT_FILL_HOLES):
        self.cfg, self.R, self.device = cfg, n_streams, device
        self.caches = [B.OvggtCache.from_stream(cfg, device=device, compaction=compaction) for _ in range(n_streams)]
        self.next_frame = [0] * n_streams
        host = [gen.frame_inputs(cfg.replace(seed=cfg.seed + seed_offset), t) for t in range(pool_frames)]
        self.host_frames = host
        self.frames = [DeviceFrame(cfg, fi, device) for fi in host]
        self.out = self.caches[0].new_out()
        self.i = 0

    def fill_frames(self) -> int:
        """Steps until every stream's cache is full, plus one more round."""
        per = -(-self.cfg.budget // self.cfg.tokens_per_frame) + 1
        return per * self.R

    def step(self, stream) -> None:
        r = self.i % self.R
        f = self.frames[self.i % len(self.frames)]
        t = self.next_frame[r]
        self.caches[r].layer_step(0, t, f.q, f.k, f.v, f.resid, f.conf, f.rho, out=self.out, stream=stream)
        self.next_frame[r] = t + 1
        self.i += 1

    def step_host(self, pinned: List[DeviceFrame], outs, stream) -> None:
        r = self.i % self.R
        f = pinned[self.i % len(pinned)]
        t = self.next_frame[r]
        self.caches[r].layer_step_host(0, t, f.q, f.k, f.v, f.resid, f.conf, f.rho, outs[self.i % len(outs)], stream=stream)
        self.next_frame[r] = t + 1
        self.i += 1

    def set_overlap(self, on: bool) -> None:
        for c in self.caches:
            c.set_overlap(on)

    def profile_enable(self, on: bool) -> None:
        for c in self.caches:
            c.profile_enable(on)

    def profile_read(self) -> dict:
        tot = None
        for c in self.caches:
            p = c.profile_read(reset=True)
            if tot is None:
                tot = p
            else:
                for k, v in p.items():
                    tot[k]["ms"] += v["ms"]
                    tot[k]["count"] += v["count"]
        return tot

    def check(self) -> None:
        for c in self.caches:
            st = c.stats(0)
            assert st["device_status"] == 0 and st["n_cached"] == self.cfg.budget, st

    def destroy(self) -> None:
        for c in self.caches:
            c.destroy()


class _Timer:
    """Accumulates device time of the regions it brackets (CUDA events on one stream)."""

    def __init__(self, stream):
        self.stream, self.pairs = stream, []

    def __call__(self, fn: Callable[[], None]) -> None:
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(self.stream)
        fn()
        b.record(self.stream)
        self.pairs.append((a, b))

    def total_ms(self) -> float:
        torch.cuda.synchronize()
        t = sum(a.elapsed_time(b) for a, b in self.pairs)
        self.pairs = []
        return t


class _Matmul:
    """x @ W of the scaffold: torch's matmul, or the library's own tcgen05 GEMM (ovggt_k_gemm_bf16).  Either way it is
    scaffold time, not the streaming step's."""

    def __init__(self, kind: str, device):
        assert kind in ("torch", "library")
        self.kind = kind
        self.status = torch.zeros(16, dtype=torch.int32, device=device)

    def __call__(self, x: torch.Tensor, w: torch.Tensor, stream=None) -> torch.Tensor:
        if self.kind == "torch":
            return x @ w
        return B.k_gemm_bf16(x.contiguous(), w, status=self.status, stream=stream)

    def check(self) -> None:
        assert int(self.status[0].item()) == 0


def _randn(shape, std, device, dtype, gen_):
    return (torch.randn(shape, generator=gen_, device=device, dtype=torch.float32) * std).to(dtype)


class ProjectionStack:
    """24 global-attention layers with their own caches.  Per layer: q, k, v = x W_qkv (random-init N(0, 0.02)),
    the library attends, x <- x + O W_o.  There is no MLP in this workload, so the residual that feeds the activation
    score is the seeded synthetic one of the single-layer workload.  `tap(t, l, q, k, v, resid)`, if given, sees every
    library input and may return priorities to rank instead of the library's own (teacher forcing in the tests);
    `after(t, l, out)` sees the attention output of every library call."""

    def __init__(self, cfg: gen.StreamConfig, device, compaction: int = B.COMPACT_FILL_HOLES, matmul: str = "library"):
        assert cfg.dtype == gen.DTYPE_BF16
        self.cfg, self.device = cfg, device
        self.mm = _Matmul(matmul, device)
        self.cache = B.OvggtCache.from_stream(cfg, device=device, compaction=compaction)
        g = torch.Generator(device=device)
        g.manual_seed(cfg.seed)
        C, L = cfg.dim, cfg.n_layers
        self.w_qkv = [_randn((C, 3 * C), 0.02, device, torch.bfloat16, g) for _ in range(L)]
        self.w_o = [_randn((C, C), 0.02, device, torch.bfloat16, g) for _ in range(L)]
        self.out = self.cache.new_out()
        self.tap: Optional[Callable] = None
        self.after: Optional[Callable] = None

    def frame(self, t: int, x: torch.Tensor, resid: List[torch.Tensor], conf: torch.Tensor, rho: float, stream,
              lib: Optional[_Timer] = None) -> torch.Tensor:
        """x: [M, C] patch embeddings of frame t (bf16).  resid[l]: the layer's synthetic residual rows."""
        C = self.cfg.dim
        for l in range(self.cfg.n_layers):
            # embeddings are N(0, 1) over 1024 columns and the weights N(0, 0.02): q, k, v come out near N(0, 0.4)
            qkv = self.mm(x, self.w_qkv[l], stream)
            q, k, v = (qkv[:, i * C:(i + 1) * C].contiguous() for i in range(3))
            ov = self.tap(t, l, q, k, v, resid[l]) if self.tap else None
            run = lambda: self.cache.layer_step(l, t, q, k, v, resid[l], conf, rho, score_override=ov, out=self.out,
                                                stream=stream)
            lib(run) if lib else run()
            if self.after:
                self.after(t, l, self.out)
            x = x + self.mm(self.out, self.w_o[l], stream)
        return x

    def destroy(self) -> None:
        self.mm.check()
        self.cache.destroy()


def _layer_norm(x: torch.Tensor) -> torch.Tensor:
    return torch.nn.functional.layer_norm(x.float(), (x.shape[-1],)).to(x.dtype)


class Aggregator:
    """Alternating aggregator: per depth a frame-attention block (attention among the frame's own tokens) and a
    global-attention block (the library: attention over the bounded cache), each followed by an MLP of width 4C,
    random-init N(0, 0.02), LayerScale taken as 1.  In the global block the library's two halves bracket the MLP:
    attend -> h = x + O W_o -> r = MLP(LN(h)) -> compress(resid = r) -> x = h + r, so the activation score sees the
    block's real MLP output.  With batched_compress the compress of all layers is deferred to the end of the frame and
    issued as one call (ovggt_layers_compress): that is the order a real model needs, whose anchor inputs (coverage,
    confidence) come out of its heads after the last block.  `tap` and `after` as in ProjectionStack."""

    def __init__(self, cfg: gen.StreamConfig, device, compaction: int = B.COMPACT_FILL_HOLES,
                 batched_compress: bool = True, frame_attention: str = "library", matmul: str = "library"):
        """frame_attention: "library" runs the attention among the frame's own tokens on the library's tcgen05 kernel
        (ovggt_k_attention with N = M: the same kernel that serves the cache); "torch" uses torch's SDPA.
        matmul: "library" runs every projection and MLP product on ovggt_k_gemm_bf16; "torch" on torch's matmul."""
        self.batched_compress = batched_compress
        self.mm = _Matmul(matmul, device)
        self.frame_attention = frame_attention
        M, H = cfg.tokens_per_frame, cfg.n_heads
        self._fa_scratch = torch.empty(B.lib().ovggt_k_attention_scratch_bytes(M, M, H), dtype=torch.uint8, device=device)
        self._fa_status = torch.zeros(16, dtype=torch.int32, device=device)
        self._fa_out = torch.empty((M, cfg.dim), dtype=torch.bfloat16, device=device)
        assert cfg.dtype == gen.DTYPE_BF16
        self.cfg, self.device = cfg, device
        self.cache = B.OvggtCache.from_stream(cfg, device=device, compaction=compaction)
        g = torch.Generator(device=device)
        g.manual_seed(cfg.seed + 1)
        C, L, bf = cfg.dim, cfg.n_layers, torch.bfloat16
        mk = lambda shape: _randn(shape, 0.02, device, bf, g)
        self.blocks = [{kind: {"qkv": mk((C, 3 * C)), "o": mk((C, C)), "fc1": mk((C, 4 * C)), "fc2": mk((4 * C, C))}
                        for kind in ("frame", "global")} for _ in range(L)]
        self.out = self.cache.new_out()
        self.tap: Optional[Callable] = None
        self.after: Optional[Callable] = None

    def _mlp(self, w, h, stream=None):
        return self.mm(torch.nn.functional.gelu(self.mm(_layer_norm(h), w["fc1"], stream)), w["fc2"], stream)

    def frame(self, t: int, x: torch.Tensor, conf: torch.Tensor, rho: float, stream,
              lib: Optional[_Timer] = None) -> torch.Tensor:
        cfg = self.cfg
        C, H, M = cfg.dim, cfg.n_heads, cfg.tokens_per_frame
        resids, overrides = [], []
        for l in range(cfg.n_layers):
            w = self.blocks[l]["frame"]
            qkv = self.mm(_layer_norm(x), w["qkv"], stream)
            if self.frame_attention == "library":
                fq, fk, fv = (qkv[:, i * C:(i + 1) * C].contiguous() for i in range(3))
                a = B.k_attention(fq, fk, fv, H, out=self._fa_out, scratch=self._fa_scratch, status=self._fa_status,
                                  stream=stream)
            else:
                q3 = qkv.view(M, 3, H, C // H).permute(1, 2, 0, 3)                               # [3, H, M, d]
                a = torch.nn.functional.scaled_dot_product_attention(q3[0], q3[1], q3[2]).permute(1, 0, 2).reshape(M, C)
            x = x + self.mm(a, w["o"], stream)
            x = x + self._mlp(w, x, stream)
            w = self.blocks[l]["global"]
            qkv = self.mm(_layer_norm(x), w["qkv"], stream)
            q, k, v = (qkv[:, i * C:(i + 1) * C].contiguous() for i in range(3))
            att = lambda: self.cache.layer_attend(l, t, q, k, v, out=self.out, stream=stream)
            lib(att) if lib else att()
            if self.after:
                self.after(t, l, self.out)
            h = x + self.mm(self.out, w["o"], stream)
            r = self._mlp(w, h, stream).contiguous()
            ov = self.tap(t, l, q, k, v, r) if self.tap else None
            if self.batched_compress:
                resids.append(r)
                overrides.append(ov)
            else:
                cmp_ = lambda: self.cache.layer_compress(l, t, r, conf, rho, score_override=ov, stream=stream)
                lib(cmp_) if lib else cmp_()
            x = h + r
        if self.batched_compress:
            ovs = overrides if any(o is not None for o in overrides) else None
            cmp_ = lambda: self.cache.layers_compress(t, resids, conf, rho, score_overrides=ovs, stream=stream)
            lib(cmp_) if lib else cmp_()
        return x

    def destroy(self) -> None:
        self.mm.check()
        self.cache.destroy()


def patch_embeddings(cfg: gen.StreamConfig, t: int, device) -> torch.Tensor:
    """Synthetic patch embeddings of frame t: N(0, 1), seeded per frame, rounded to bf16."""
    rng = np.random.Generator(np.random.Philox(key=[np.uint64(cfg.seed), np.uint64((t << 8) | 0x40)]))
    x = rng.standard_normal((cfg.tokens_per_frame, cfg.dim), dtype=np.float32)
    return torch.from_numpy(x).to(torch.bfloat16).to(device)


def frame_side_inputs(cfg: gen.StreamConfig, t: int, device, layers_with_resid: int = 0):
    """(conf, rho, [resid per layer]) of frame t: the per-frame anchor inputs, and synthetic residual rows for the
    workloads that have no MLP of their own."""
    fi = gen.frame_inputs(cfg, t, fields=("anchor inputs only",))
    conf = torch.from_numpy(fi.conf).to(device)
    resid = []
    for l in range(layers_with_resid):
        r = gen.frame_inputs(cfg, t, layer=l, fields=("resid",)).resid
        resid.append(torch.from_numpy(r).to(torch.bfloat16).to(device))
    return conf, fi.rho, resid


def time_per_step(fn: Callable[[], None], steps: int, stream):
    """(total ms, per-step ms array) of `steps` calls of fn, device time between consecutive events on `stream`."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record(stream)
    for i in range(steps):
        fn()
        ev[i + 1].record(stream)
    torch.cuda.synchronize()
    per = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(steps)])
    return ev[0].elapsed_time(ev[steps]), per


def flatness(per_step: np.ndarray) -> dict:
    k = len(per_step)
    slope = float(np.polyfit(np.arange(k), per_step, 1)[0]) if k >= 3 else 0.0
    return {"median": float(np.median(per_step)), "max": float(per_step.max()), "min": float(per_step.min()),
            "slope_ms_per_frame": slope, "max_over_median": float(per_step.max() / np.median(per_step)),
            "second_half_median": float(np.median(per_step[k // 2:]))}


def attention_flops(M: int, N: int, C: int) -> float:
    return 4.0 * M * N * C
