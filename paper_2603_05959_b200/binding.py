"""Thin ctypes binding of libovggt.so (the C ABI of include/ovggt.h): argument marshalling only.

Every step of the hot path runs in the library's CUDA kernels; torch is used for device memory,
streams and nothing else.  If the library is missing the import fails loudly - there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# OVGGT_LIBRARY=checked selects the build with range-checked indices (paper_2603_05959_b200/build.py --checked)
LIB_PATH = os.path.join(_HERE, "libovggt_checked.so" if os.environ.get("OVGGT_LIBRARY") == "checked" else "libovggt.so")
MAX_ANCHORS = 16

DTYPE_F32, DTYPE_BF16 = 0, 1
SCORE_HYBRID, SCORE_RESIDUAL_STORED, SCORE_RANDOM, SCORE_QK, SCORE_ATTN = 0, 1, 2, 3, 4
FLAG_EVICTABLE, FLAG_INIT, FLAG_HIST = 0, 1, 2
COMPACT_FILL_HOLES, COMPACT_STABLE_GATHER = 0, 1
PROF_CLASSES = ["append", "attention", "row_norms", "diversity", "select", "compact"]

EXPORTED = [
    "ovggt_workspace_bytes", "ovggt_cache_create", "ovggt_cache_destroy", "ovggt_layer_attend",
    "ovggt_layer_compress", "ovggt_layers_compress", "ovggt_layer_step", "ovggt_layer_step_host", "ovggt_cache_stats",
    "ovggt_cache_export", "ovggt_cache_import", "ovggt_cache_reset", "ovggt_cache_anchor_decision",
    "ovggt_camera_compress", "ovggt_cache_selftest_bounded_wait", "ovggt_cache_clear_status", "ovggt_cache_last_selection", "ovggt_kernel_launches",
    "ovggt_cache_profile_enable", "ovggt_cache_profile_read", "ovggt_cache_set_overlap", "ovggt_cache_set_key_bound",
    "ovggt_strerror", "ovggt_last_cuda_error", "ovggt_k_row_norms", "ovggt_k_diversity_scratch_bytes",
    "ovggt_k_diversity", "ovggt_k_diversity_static", "ovggt_k_select", "ovggt_k_compact", "ovggt_k_attention_scratch_bytes",
    "ovggt_k_attention", "ovggt_k_key_norm_bound", "ovggt_k_attention_bounded", "ovggt_k_gemm_bf16",
]


class OvggtConfig(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
        ("n_special", C.c_int32), ("grid_h", C.c_int32), ("grid_w", C.c_int32),
        ("budget", C.POINTER(C.c_int32)),
        ("anchor_tokens", C.c_int32), ("k_max", C.c_int32), ("min_anchor_interval", C.c_int32),
        ("tau", C.c_float), ("alpha", C.c_float), ("beta", C.c_float),
        ("protect_first_frame", C.c_int32), ("score_mode", C.c_int32), ("dtype", C.c_int32),
        ("compaction", C.c_int32), ("random_seed", C.c_uint64), ("camera_head", C.c_int32),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
    ]


class OvggtFrameIO(C.Structure):
    _fields_ = [
        ("frame_id", C.c_int64),
        ("q", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p), ("resid", C.c_void_p),
        ("conf", C.c_void_p), ("rho", C.c_float), ("score_override", C.c_void_p), ("out", C.c_void_p),
    ]


class OvggtStats(C.Structure):
    _fields_ = [
        ("n_cached", C.c_int32), ("n_protected_init", C.c_int32), ("n_protected_hist", C.c_int32),
        ("n_active_anchors", C.c_int32), ("anchor_frames", C.c_int64 * MAX_ANCHORS),
        ("frames_seen", C.c_int64), ("evicted_total", C.c_int64),
        ("last_n_candidates", C.c_int32), ("last_n_survivors", C.c_int32),
        ("bytes_resident", C.c_uint64), ("device_status", C.c_int32),
    ]


ERR_TIMEOUT, ERR_UNSUPPORTED, ERR_TOO_LARGE = -9, -10, -11      # (the codes of include/ovggt.h that callers test for)


class OvggtError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().ovggt_strerror(code).decode()
        extra = f" (cuda error {lib().ovggt_last_cuda_error()})" if code == -7 else ""
        super().__init__(f"{where}: {msg}{extra} [{code}]")


_LIB = None


def lib():
    """Load libovggt.so; raises if it has not been built (python -m paper_2603_05959_b200.build)."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with paper_2603_05959_b200/build.py; "
                              "there is no CPU or PyTorch fallback")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.ovggt_workspace_bytes.restype = C.c_size_t
        L.ovggt_workspace_bytes.argtypes = [C.POINTER(OvggtConfig)]
        L.ovggt_cache_create.argtypes = [C.POINTER(OvggtConfig), C.POINTER(vp)]
        L.ovggt_cache_destroy.argtypes = [vp]
        for name in ("ovggt_layer_attend", "ovggt_layer_compress", "ovggt_layers_compress", "ovggt_layer_step", "ovggt_layer_step_host"):
            getattr(L, name).argtypes = [vp, i32, C.POINTER(OvggtFrameIO), vp]
        L.ovggt_layers_compress.argtypes = [vp, C.POINTER(OvggtFrameIO), i32, vp]
        L.ovggt_cache_stats.argtypes = [vp, i32, C.POINTER(OvggtStats)]
        L.ovggt_cache_export.argtypes = [vp, i32, vp, vp, vp, vp, vp, C.POINTER(i32)]
        L.ovggt_cache_import.argtypes = [vp, i32, vp, vp, vp, vp, vp, i32, i64, i64]
        L.ovggt_cache_reset.argtypes = [vp]
        L.ovggt_cache_clear_status.argtypes = [vp]
        L.ovggt_cache_selftest_bounded_wait.argtypes = [vp, C.c_uint32, C.POINTER(C.c_uint64), vp]
        L.ovggt_cache_anchor_decision.argtypes = [vp, i64, C.POINTER(i32), C.POINTER(i64)]
        L.ovggt_camera_compress.argtypes = [vp, i32, C.POINTER(OvggtFrameIO), i32, i64, vp]
        L.ovggt_cache_last_selection.argtypes = [vp, i32, vp, C.POINTER(i32), vp, C.POINTER(i32)]
        L.ovggt_cache_profile_enable.argtypes = [vp, i32]
        L.ovggt_cache_set_overlap.argtypes = [vp, i32]
        L.ovggt_cache_set_key_bound.argtypes = [vp, i32]
        L.ovggt_cache_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64), i32]
        L.ovggt_kernel_launches.restype = C.c_uint64
        L.ovggt_strerror.restype = C.c_char_p
        L.ovggt_strerror.argtypes = [C.c_int]
        L.ovggt_k_row_norms.argtypes = [vp, i32, i32, i32, vp, vp]
        L.ovggt_k_diversity_scratch_bytes.restype = C.c_size_t
        L.ovggt_k_diversity_scratch_bytes.argtypes = [i32, i32]
        L.ovggt_k_diversity.argtypes = [vp, i32, i32, i32, vp, vp, vp]
        L.ovggt_k_diversity_static.argtypes = [vp, i32, i32, i32, vp, vp]
        L.ovggt_k_select.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
        L.ovggt_k_compact.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp]
        L.ovggt_k_attention_scratch_bytes.restype = C.c_size_t
        L.ovggt_k_attention_scratch_bytes.argtypes = [i32, i32, i32]
        L.ovggt_k_attention.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp]
        L.ovggt_k_key_norm_bound.argtypes = [vp, i32, i32, vp, vp]
        L.ovggt_k_gemm_bf16.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
        L.ovggt_k_attention_bounded.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp]
        _LIB = L
    return _LIB


def _check(code: int, where: str) -> None:
    if code != 0:
        raise OvggtError(code, where)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _dptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous()
    return t.data_ptr()


def torch_dtype(dtype: int) -> torch.dtype:
    return torch.float32 if dtype == DTYPE_F32 else torch.bfloat16


def kernel_launches() -> int:
    return int(lib().ovggt_kernel_launches())


# ------------------------------------------------------------------ the cache handle

class OvggtCache:
    """ovggt_cache_create / ovggt_layer_step / ovggt_cache_stats / ovggt_cache_destroy.

    The workspace is one torch uint8 tensor on the current CUDA device, allocated here and handed to
    the library, which lays all per-layer buffers out inside it.
    """

    def __init__(self, *, n_layers=1, n_heads=16, head_dim=64, n_special=5, grid_h=37, grid_w=37,
                 budget=16384, anchor_tokens=64, k_max=3, min_anchor_interval=100, tau=0.2, alpha=0.5,
                 beta=0.5, protect_first_frame=1, score_mode=SCORE_HYBRID, dtype=DTYPE_BF16,
                 compaction=COMPACT_FILL_HOLES, random_seed=0, camera_head=0,
                 device: Optional[torch.device] = None):
        budgets = [budget] * n_layers if isinstance(budget, int) else list(budget)
        assert len(budgets) == n_layers
        self._budgets = (C.c_int32 * n_layers)(*budgets)
        self.cfg = OvggtConfig(n_layers, n_heads, head_dim, n_special, grid_h, grid_w, self._budgets,
                               anchor_tokens, k_max, min_anchor_interval, tau, alpha, beta,
                               protect_first_frame, score_mode, dtype, compaction, random_seed, camera_head, None, 0)
        self.compaction = compaction
        self.M = n_special + grid_h * grid_w
        self.C = n_heads * head_dim
        self.n_patches = grid_h * grid_w
        self.dtype = dtype
        self.budgets = budgets
        need = lib().ovggt_workspace_bytes(C.byref(self.cfg))
        if need == 0:
            # let create report the precise reason
            self.cfg.workspace, self.cfg.workspace_bytes = 1024, 0
            h = C.c_void_p()
            _check(lib().ovggt_cache_create(C.byref(self.cfg), C.byref(h)), "ovggt_cache_create")
            raise OvggtError(-1, "ovggt_cache_create")
        self.device = device or torch.device("cuda", torch.cuda.current_device())
        self.workspace = torch.empty(need + 1024, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        self.cfg.workspace, self.cfg.workspace_bytes = base, need
        self.workspace_bytes = need
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(lib().ovggt_cache_create(C.byref(self.cfg), C.byref(h)), "ovggt_cache_create")
        self._h = h

    @classmethod
    def from_stream(cls, cfg, **over) -> "OvggtCache":
        kw = dict(n_layers=cfg.n_layers, n_heads=cfg.n_heads, head_dim=cfg.head_dim,
                  n_special=cfg.n_special, grid_h=cfg.grid_h, grid_w=cfg.grid_w, budget=cfg.budget,
                  anchor_tokens=cfg.anchor_tokens, k_max=cfg.k_max,
                  min_anchor_interval=cfg.min_anchor_interval, tau=cfg.tau, alpha=cfg.alpha,
                  beta=cfg.beta, protect_first_frame=cfg.protect_first_frame,
                  score_mode=cfg.score_mode, dtype=cfg.dtype, random_seed=cfg.seed)
        kw.update(over)
        return cls(**kw)

    def destroy(self) -> None:
        if getattr(self, "_h", None):
            lib().ovggt_cache_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def _io(self, frame_id, q=None, k=None, v=None, resid=None, conf=None, rho=float("nan"),
            score_override=None, out=None, host=False) -> OvggtFrameIO:
        ptr = (lambda t: None if t is None else t.data_ptr()) if host else _dptr
        return OvggtFrameIO(int(frame_id), ptr(q), ptr(k), ptr(v), ptr(resid), ptr(conf), float(rho),
                            ptr(score_override), ptr(out))

    def new_out(self) -> torch.Tensor:
        return torch.empty((self.M, self.C), dtype=torch_dtype(self.dtype), device=self.device)

    def layer_attend(self, layer, frame_id, q, k, v, out=None, stream=None) -> torch.Tensor:
        out = self.new_out() if out is None else out
        io = self._io(frame_id, q=q, k=k, v=v, out=out)
        _check(lib().ovggt_layer_attend(self._h, layer, C.byref(io), _stream_ptr(stream)), "ovggt_layer_attend")
        return out

    def layer_compress(self, layer, frame_id, resid, conf=None, rho=float("nan"), score_override=None,
                       stream=None) -> None:
        io = self._io(frame_id, resid=resid, conf=conf, rho=rho, score_override=score_override)
        _check(lib().ovggt_layer_compress(self._h, layer, C.byref(io), _stream_ptr(stream)), "ovggt_layer_compress")

    def layers_compress(self, frame_id, resids, conf=None, rho=float("nan"), score_overrides=None, stream=None) -> None:
        """ovggt_layers_compress: resids[l] (and optionally score_overrides[l]) per layer, one call for all layers."""
        n = len(resids)
        ios = (OvggtFrameIO * n)()
        for l in range(n):
            ov = None if score_overrides is None else score_overrides[l]
            ios[l] = self._io(frame_id, resid=resids[l], conf=conf, rho=rho, score_override=ov)
        _check(lib().ovggt_layers_compress(self._h, ios, n, _stream_ptr(stream)), "ovggt_layers_compress")

    def anchor_decision(self, frame_id):
        """(registered, demoted_frame) of frame_id as this (aggregator) handle decided it."""
        reg, dem = C.c_int32(0), C.c_int64(-1)
        _check(lib().ovggt_cache_anchor_decision(self._h, int(frame_id), C.byref(reg), C.byref(dem)),
               "ovggt_cache_anchor_decision")
        return bool(reg.value), int(dem.value)

    def camera_compress(self, layer, frame_id, resid, registered, demoted_frame, score_override=None, stream=None) -> None:
        io = self._io(frame_id, resid=resid, score_override=score_override)
        _check(lib().ovggt_camera_compress(self._h, layer, C.byref(io), int(bool(registered)), int(demoted_frame),
                                           _stream_ptr(stream)), "ovggt_camera_compress")

    @classmethod
    def camera(cls, *, n_layers=1, n_heads=16, head_dim=64, budget=144, k_max=3, beta=0.5, protect_first_frame=1,
               score_mode=SCORE_HYBRID, dtype=DTYPE_BF16, **kw) -> "OvggtCache":
        """The camera head's cache (Supp. C): one token per frame."""
        return cls(n_layers=n_layers, n_heads=n_heads, head_dim=head_dim, n_special=1, grid_h=0, grid_w=0,
                   budget=budget, anchor_tokens=0, k_max=k_max, beta=beta, protect_first_frame=protect_first_frame,
                   score_mode=score_mode, dtype=dtype, camera_head=1, **kw)

    def layer_step(self, layer, frame_id, q, k, v, resid, conf=None, rho=float("nan"), score_override=None,
                   out=None, stream=None) -> torch.Tensor:
        out = self.new_out() if out is None else out
        io = self._io(frame_id, q, k, v, resid, conf, rho, score_override, out)
        _check(lib().ovggt_layer_step(self._h, layer, C.byref(io), _stream_ptr(stream)), "ovggt_layer_step")
        return out

    def layer_step_host(self, layer, frame_id, q, k, v, resid, conf, rho, out, stream=None) -> None:
        """All tensors are host (ideally pinned) torch tensors; the copies run inside the call."""
        io = self._io(frame_id, q, k, v, resid, conf, rho, None, out, host=True)
        _check(lib().ovggt_layer_step_host(self._h, layer, C.byref(io), _stream_ptr(stream)), "ovggt_layer_step_host")

    def stats(self, layer=0) -> dict:
        st = OvggtStats()
        code = lib().ovggt_cache_stats(self._h, layer, C.byref(st))
        d = {name: getattr(st, name) for name, _ in OvggtStats._fields_ if name != "anchor_frames"}
        d["anchor_frames"] = [int(st.anchor_frames[i]) for i in range(st.n_active_anchors)]
        _check(code, "ovggt_cache_stats")
        return d

    def export(self, layer=0, with_kv=True) -> dict:
        n = C.c_int32(0)
        _check(lib().ovggt_cache_export(self._h, layer, None, None, None, None, None, C.byref(n)), "ovggt_cache_export")
        n = n.value
        ids = np.empty(n, np.int64); flags = np.empty(n, np.uint8); scores = np.empty(n, np.float32)
        el = np.float32 if self.dtype == DTYPE_F32 else np.uint16
        k = np.empty((n, self.C), el) if with_kv else None
        v = np.empty((n, self.C), el) if with_kv else None
        p = lambda a: None if a is None else a.ctypes.data
        _check(lib().ovggt_cache_export(self._h, layer, p(ids), p(flags), p(scores), p(k), p(v), None), "ovggt_cache_export")
        return {"ids": ids, "flags": flags, "stored": scores, "k": k, "v": v}

    def import_(self, layer, ids, flags, scores, k, v, next_frame_id, last_registration_frame) -> None:
        ids = np.ascontiguousarray(ids, np.int64); flags = np.ascontiguousarray(flags, np.uint8)
        scores = np.ascontiguousarray(scores, np.float32)
        k = np.ascontiguousarray(k); v = np.ascontiguousarray(v)
        _check(lib().ovggt_cache_import(self._h, layer, ids.ctypes.data, flags.ctypes.data, scores.ctypes.data,
                                        k.ctypes.data, v.ctypes.data, len(ids), int(next_frame_id),
                                        int(last_registration_frame)), "ovggt_cache_import")

    def selftest_bounded_wait(self, limit_us: int, stream=None) -> int:
        """Runs the library's bounded device-side wait on a barrier nothing completes; returns the nanoseconds it
        waited.  The handle's status word then holds the time-out code until clear_status()."""
        ns = C.c_uint64(0)
        _check(lib().ovggt_cache_selftest_bounded_wait(self._h, int(limit_us), C.byref(ns), _stream_ptr(stream)),
               "ovggt_cache_selftest_bounded_wait")
        return int(ns.value)

    def clear_status(self) -> None:
        _check(lib().ovggt_cache_clear_status(self._h), "ovggt_cache_clear_status")

    def reset(self) -> None:
        _check(lib().ovggt_cache_reset(self._h), "ovggt_cache_reset")

    def set_key_bound(self, on: bool) -> None:
        _check(lib().ovggt_cache_set_key_bound(self._h, int(on)), "ovggt_cache_set_key_bound")

    def set_overlap(self, on: bool) -> None:
        _check(lib().ovggt_cache_set_overlap(self._h, int(on)), "ovggt_cache_set_overlap")

    def profile_enable(self, on: bool) -> None:
        _check(lib().ovggt_cache_profile_enable(self._h, int(on)), "ovggt_cache_profile_enable")

    def profile_read(self, reset: bool = True) -> dict:
        ms = (C.c_double * len(PROF_CLASSES))()
        cnt = (C.c_int64 * len(PROF_CLASSES))()
        _check(lib().ovggt_cache_profile_read(self._h, ms, cnt, int(reset)), "ovggt_cache_profile_read")
        return {name: {"ms": ms[i], "count": int(cnt[i])} for i, name in enumerate(PROF_CLASSES)}

    def last_selection(self, layer=0) -> dict:
        nc, ns = C.c_int32(0), C.c_int32(0)
        _check(lib().ovggt_cache_last_selection(self._h, layer, None, C.byref(nc), None, C.byref(ns)),
               "ovggt_cache_last_selection")
        r = np.empty(nc.value, np.float32); s = np.empty(ns.value, np.int32)
        _check(lib().ovggt_cache_last_selection(self._h, layer, r.ctypes.data, None, s.ctypes.data, None),
               "ovggt_cache_last_selection")
        return {"r": r, "survivors": s}


# ------------------------------------------------------------------ single kernels

def k_row_norms(x: torch.Tensor, stream=None) -> torch.Tensor:
    dtype = DTYPE_F32 if x.dtype == torch.float32 else DTYPE_BF16
    s = torch.empty(x.shape[0], dtype=torch.float32, device=x.device)
    _check(lib().ovggt_k_row_norms(_dptr(x), x.shape[0], x.shape[1], dtype, _dptr(s), _stream_ptr(stream)),
           "ovggt_k_row_norms")
    return s


def k_diversity(K: torch.Tensor, stream=None) -> torch.Tensor:
    dtype = DTYPE_F32 if K.dtype == torch.float32 else DTYPE_BF16
    d = torch.empty(K.shape[0], dtype=torch.float32, device=K.device)
    scratch = torch.empty(lib().ovggt_k_diversity_scratch_bytes(K.shape[0], K.shape[1]), dtype=torch.uint8,
                          device=K.device)
    _check(lib().ovggt_k_diversity(_dptr(K), K.shape[0], K.shape[1], dtype, _dptr(d), _dptr(scratch),
                                   _stream_ptr(stream)), "ovggt_k_diversity")
    return d


def k_diversity_static(K: torch.Tensor, d: torch.Tensor, stream=None) -> torch.Tensor:
    """ovggt_k_diversity_static: the caller passes the input K and the output d only; the scratch is an array
    built into the library, so the call allocates nothing (d is given, not created here)."""
    dtype = DTYPE_F32 if K.dtype == torch.float32 else DTYPE_BF16
    _check(lib().ovggt_k_diversity_static(_dptr(K), K.shape[0], K.shape[1], dtype, _dptr(d), _stream_ptr(stream)),
           "ovggt_k_diversity_static")
    return d


def k_select(r: torch.Tensor, flags: torch.Tensor, budget: int, stream=None) -> torch.Tensor:
    """r [batch, N] or [N] fp32, flags same shape uint8 -> survivors [batch, min(N, B)] int32."""
    r2 = r.view(1, -1) if r.dim() == 1 else r
    f2 = flags.view(1, -1) if flags.dim() == 1 else flags
    batch, N = r2.shape
    out = torch.empty((batch, min(N, budget)), dtype=torch.int32, device=r.device)
    scratch = torch.empty(4 * N * batch + 64, dtype=torch.uint8, device=r.device)
    _check(lib().ovggt_k_select(_dptr(r2), _dptr(f2), N, int(budget), batch, _dptr(out), _dptr(scratch),
                                _stream_ptr(stream)), "ovggt_k_select")
    return out if r.dim() == 2 else out[0]


def k_compact(k_src, v_src, survivors, k_dst=None, v_dst=None, stream=None):
    dtype = DTYPE_F32 if k_src.dtype == torch.float32 else DTYPE_BF16
    n_keep, Cdim = survivors.shape[0], k_src.shape[1]
    k_dst = torch.empty((n_keep, Cdim), dtype=k_src.dtype, device=k_src.device) if k_dst is None else k_dst
    v_dst = torch.empty((n_keep, Cdim), dtype=k_src.dtype, device=k_src.device) if v_dst is None else v_dst
    _check(lib().ovggt_k_compact(_dptr(k_src), _dptr(v_src), _dptr(survivors), n_keep, Cdim, dtype,
                                 _dptr(k_dst), _dptr(v_dst), _stream_ptr(stream)), "ovggt_k_compact")
    return k_dst, v_dst


def k_gemm_bf16(a: torch.Tensor, b: torch.Tensor, out=None, status=None, stream=None) -> torch.Tensor:
    """out [M, N] = a [M, K] @ b [K, N], bf16 in and out, on the library's tcgen05 GEMM."""
    assert a.dtype == torch.bfloat16 and b.dtype == torch.bfloat16 and a.shape[1] == b.shape[0]
    M, K = a.shape
    N = b.shape[1]
    out = torch.empty((M, N), dtype=torch.bfloat16, device=a.device) if out is None else out
    own = status is None
    if own:
        status = torch.zeros(16, dtype=torch.int32, device=a.device)
    _check(lib().ovggt_k_gemm_bf16(_dptr(a), _dptr(b), M, N, K, _dptr(out), _dptr(status), _stream_ptr(stream)),
           "ovggt_k_gemm_bf16")
    if own:
        _check(int(status[0].item()), "ovggt_k_gemm_bf16 (device status)")
    return out


def k_key_norm_bound(k: torch.Tensor, n_heads: int, stream=None) -> torch.Tensor:
    """[n_heads] fp32: the largest squared norm of any key's 64 columns of each head (bf16 keys)."""
    out = torch.empty(n_heads, dtype=torch.float32, device=k.device)
    _check(lib().ovggt_k_key_norm_bound(_dptr(k), k.shape[0], n_heads, _dptr(out), _stream_ptr(stream)),
           "ovggt_k_key_norm_bound")
    return out


def k_attention(q, k, v, n_heads: int, out=None, scratch=None, status=None, stream=None, bounded=False) -> torch.Tensor:
    """bounded: bf16 only - first compute the key-norm bound, then attend with the fixed softmax reference."""
    dtype = DTYPE_F32 if q.dtype == torch.float32 else DTYPE_BF16
    M, N = q.shape[0], k.shape[0]
    out = torch.empty_like(q) if out is None else out
    if bounded:
        assert dtype == DTYPE_BF16
        kmax2 = k_key_norm_bound(k, n_heads, stream)
        scratch = torch.empty(lib().ovggt_k_attention_scratch_bytes(M, N, n_heads), dtype=torch.uint8, device=q.device)
        st = torch.zeros(16, dtype=torch.int32, device=q.device)
        _check(lib().ovggt_k_attention_bounded(_dptr(q), _dptr(k), _dptr(v), M, N, n_heads, _dptr(out), _dptr(scratch),
                                               _dptr(st), _dptr(kmax2), _stream_ptr(stream)), "ovggt_k_attention_bounded")
        _check(int(st[0].item()), "ovggt_k_attention_bounded (device status)")
        return out
    if scratch is None:
        scratch = torch.empty(lib().ovggt_k_attention_scratch_bytes(M, N, n_heads), dtype=torch.uint8, device=q.device)
    own_status = status is None
    if own_status:
        status = torch.zeros(16, dtype=torch.int32, device=q.device)
    _check(lib().ovggt_k_attention(_dptr(q), _dptr(k), _dptr(v), M, N, n_heads, dtype, _dptr(out), _dptr(scratch),
                                   _dptr(status), _stream_ptr(stream)), "ovggt_k_attention")
    if own_status:
        code = int(status[0].item())
        _check(code, "ovggt_k_attention (device status)")
    return out
