"""Seeded synthetic input streams for the OVGGT streaming global-attention step.

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the method's arithmetic: it only draws random numbers and describes
workload shapes.  Every tensor of frame ``t`` is drawn from a counter-based
generator (numpy's Philox) keyed by ``(seed, layer, frame, tensor tag)``, so a
frame can be regenerated in isolation and both sides consume identical bits.

Workload shapes follow the paper's token layout (Sec. 3.1: ``M = 1 + 4 + N_p``
tokens per frame, ``N_p = H_p * W_p`` patches) and its hyper-parameters
(Sec. 4, Implementation Details: alpha, beta, tau, the 100-frame anchor
interval, K_max).  No dataset of the paper is used; the streams stand in for
them by shape only.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np

TAG_Q, TAG_K, TAG_V, TAG_RESID, TAG_GAIN, TAG_CONF, TAG_RHO = range(1, 8)

DTYPE_F32 = 0
DTYPE_BF16 = 1

SCORE_HYBRID = 0
SCORE_RESIDUAL_STORED = 1
SCORE_RANDOM = 2
SCORE_QK = 3
SCORE_ATTN = 4


@dataclasses.dataclass(frozen=True)
class StreamConfig:
    """One synthetic workload: token layout, cache budget, anchor rule, input recipe."""

    name: str
    n_layers: int = 1
    n_heads: int = 16
    head_dim: int = 64
    n_special: int = 5
    grid_h: int = 37
    grid_w: int = 37
    budget: int = 16384
    anchor_tokens: int = 64
    k_max: int = 3
    min_anchor_interval: int = 100
    tau: float = 0.2
    alpha: float = 0.5
    beta: float = 0.5
    protect_first_frame: int = 1
    score_mode: int = SCORE_HYBRID
    dtype: int = DTYPE_BF16
    n_frames: int = 200
    gain_sigma: float = 0.75
    gain_mu_drift_per_1000: float = 0.0
    seed: int = 20260305

    @property
    def dim(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def n_patches(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def tokens_per_frame(self) -> int:
        return self.n_special + self.n_patches

    @property
    def max_rows(self) -> int:
        """Rows of one cache buffer: the budget plus the frame being appended."""
        return self.budget + self.tokens_per_frame

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == DTYPE_F32 else 2

    def replace(self, **kw) -> "StreamConfig":
        return dataclasses.replace(self, **kw)


def config_tiny() -> StreamConfig:
    """Tiny fp32 single layer: 4 heads x 64, 8x8 patches + 5, 16 frames, budget 256, 8 anchor tokens."""
    return StreamConfig(name="c1_tiny_fp32", n_heads=4, grid_h=8, grid_w=8, budget=256,
                        anchor_tokens=8, min_anchor_interval=4, dtype=DTYPE_F32,
                        n_frames=16, gain_sigma=0.5)


def config_vggt_layer() -> StreamConfig:
    """One VGGT-shaped global-attention layer, bf16: 16 x 64, 37x37 + 5 = 1374 tokens, budget 16384."""
    return StreamConfig(name="c2_vggt_layer_bf16")


def config_stack24() -> StreamConfig:
    """24 global-attention layers, each with its own cache of 8192 tokens, 500 frames."""
    return StreamConfig(name="c3_stack24_bf16", n_layers=24, budget=8192, n_frames=500)


def config_aggregator() -> StreamConfig:
    """518x392 frames -> 37x28 patches + 5 = 1041 tokens; budget 12288; 1000 frames."""
    return StreamConfig(name="c4_aggregator_bf16", n_layers=24, grid_h=28, grid_w=37,
                        budget=12288, n_frames=1000)


def config_ultra_long(budget: int = 16384, anchor_tokens: int = 64,
                      score_mode: int = SCORE_HYBRID) -> StreamConfig:
    """10,000-frame stress stream with the residual gain drifting by +0.1 (log-mean) per 1000 frames."""
    return StreamConfig(name=f"c5_ultra_long_b{budget}_a{anchor_tokens}", budget=budget,
                        anchor_tokens=anchor_tokens, n_frames=10000,
                        gain_mu_drift_per_1000=0.1, score_mode=score_mode)


# --------------------------------------------------------------------------- rounding helpers

def bf16_round_bits(x: np.ndarray) -> np.ndarray:
    """float32 array -> uint16 array of bfloat16 bit patterns, round-to-nearest-even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    out = (r >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """uint16 bfloat16 bit patterns -> the float32 values they denote (exact)."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_dtype(x: np.ndarray, dtype: int) -> np.ndarray:
    """float32 values representable in the configured storage type."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == DTYPE_F32:
        return x
    return bf16_bits_to_f32(bf16_round_bits(x))


# --------------------------------------------------------------------------- generators

def _rng(seed: int, layer: int, frame: int, tag: int) -> np.random.Generator:
    key = [np.uint64(seed), np.uint64((layer << 48) | (frame << 8) | tag)]
    return np.random.Generator(np.random.Philox(key=key))


@dataclasses.dataclass
class FrameInputs:
    """Inputs of one (frame, layer) step.  The float32 arrays hold values already
    rounded to the stream's storage type, so converting them to that type is exact."""

    frame_id: int
    layer: int
    q: np.ndarray        # [M, C] float32
    k: np.ndarray        # [M, C] float32
    v: np.ndarray        # [M, C] float32
    resid: np.ndarray    # [M, C] float32  (the block's FFN residual rows, LayerScale included)
    conf: np.ndarray     # [N_p]  float32  (per-patch confidence of this frame)
    rho: float           # coverage ratio of the most recent anchor in this view

    def storage(self, name: str, dtype: int) -> np.ndarray:
        """The tensor as the bytes the library receives: float32, or uint16 bf16 bit patterns."""
        x = getattr(self, name)
        return x if dtype == DTYPE_F32 else bf16_round_bits(x)


def gain_log_mean(cfg: StreamConfig, frame: int) -> float:
    return cfg.gain_mu_drift_per_1000 * float(frame // 1000)


def frame_inputs(cfg: StreamConfig, frame: int, layer: int = 0,
                 fields: Optional[tuple] = None) -> FrameInputs:
    """Draw the inputs of ``frame`` at ``layer``.

    q, k, v ~ N(0, 1); resid[j, :] = g_j * z_j with z ~ N(0, I) and
    g_j ~ lognormal(mu_t, gain_sigma) so that residual norms spread out;
    conf ~ U(0, 1) per patch and rho ~ U(0, 1) (both shared by all layers of a frame).
    """
    M, C = cfg.tokens_per_frame, cfg.dim
    want = fields or ("q", "k", "v", "resid")
    out = {}
    for name, tag in (("q", TAG_Q), ("k", TAG_K), ("v", TAG_V)):
        if name in want:
            x = _rng(cfg.seed, layer, frame, tag).standard_normal((M, C), dtype=np.float32)
            out[name] = round_to_dtype(x, cfg.dtype)
        else:
            out[name] = None
    if "resid" in want:
        z = _rng(cfg.seed, layer, frame, TAG_RESID).standard_normal((M, C), dtype=np.float32)
        g = _rng(cfg.seed, layer, frame, TAG_GAIN).lognormal(
            gain_log_mean(cfg, frame), cfg.gain_sigma, size=(M, 1)).astype(np.float32)
        out["resid"] = round_to_dtype(z * g, cfg.dtype)
    else:
        out["resid"] = None
    conf = _rng(cfg.seed, 0, frame, TAG_CONF).random(cfg.n_patches, dtype=np.float32)
    rho = float(_rng(cfg.seed, 0, frame, TAG_RHO).random())
    return FrameInputs(frame, layer, out["q"], out["k"], out["v"], out["resid"], conf, rho)
