"""Plumbing between the seeded input generator and the library: host arrays -> torch tensors."""
from __future__ import annotations

import numpy as np
import torch

from . import inputs as gen
from .binding import torch_dtype


def to_torch(x: np.ndarray, dtype: int, device=None, pin: bool = False) -> torch.Tensor:
    """float32 values that are exactly representable in `dtype` -> a tensor of that dtype."""
    t = torch.from_numpy(np.ascontiguousarray(x)).to(torch_dtype(dtype))
    if device is not None:
        return t.to(device)
    return t.pin_memory() if pin else t


class DeviceFrame:
    """The tensors of one (frame, layer) step on the device (or pinned on the host)."""

    def __init__(self, cfg: gen.StreamConfig, fi: gen.FrameInputs, device=None, pin: bool = False):
        self.frame_id = fi.frame_id
        self.rho = fi.rho
        if device is None and pin:
            # one pinned block [q | k | v | resid]: the host-buffer entry point then moves it with a single copy
            block = torch.empty((4,) + fi.q.shape, dtype=torch_dtype(cfg.dtype)).pin_memory()
            for i, x in enumerate((fi.q, fi.k, fi.v, fi.resid)):
                block[i].copy_(to_torch(x, cfg.dtype))
            self.block = block
            self.q, self.k, self.v, self.resid = block[0], block[1], block[2], block[3]
        else:
            self.q = to_torch(fi.q, cfg.dtype, device, pin)
            self.k = to_torch(fi.k, cfg.dtype, device, pin)
            self.v = to_torch(fi.v, cfg.dtype, device, pin)
            self.resid = to_torch(fi.resid, cfg.dtype, device, pin)
        conf = torch.from_numpy(fi.conf)
        self.conf = conf.to(device) if device is not None else (conf.pin_memory() if pin else conf)


def out_to_f32(out: torch.Tensor) -> np.ndarray:
    return out.detach().float().cpu().numpy()


def storage_to_f32(a: np.ndarray, dtype: int) -> np.ndarray:
    """Exported K/V rows (float32, or uint16 bf16 bit patterns) -> float32 values."""
    return a if dtype == gen.DTYPE_F32 else gen.bf16_bits_to_f32(a)
