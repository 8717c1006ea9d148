"""ctypes access to the CPU oracle (oracle/liboracle.so).  TEST INFRASTRUCTURE ONLY:
imported by the tests, the smoke check and the benchmark's CPU-baseline leg, never
by the product path."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


class OrcConfig(C.Structure):
    _fields_ = [
        ("n_heads", C.c_int32), ("head_dim", C.c_int32),
        ("n_special", C.c_int32), ("grid_h", C.c_int32), ("grid_w", C.c_int32),
        ("budget", C.c_int32), ("anchor_tokens", C.c_int32),
        ("k_max", C.c_int32), ("min_anchor_interval", C.c_int32),
        ("tau", C.c_double), ("alpha", C.c_double), ("beta", C.c_double),
        ("protect_first_frame", C.c_int32), ("score_mode", C.c_int32),
        ("diversity_per_head", C.c_int32), ("camera_cache", C.c_int32), ("random_seed", C.c_uint64),
    ]


SCORE_HYBRID, SCORE_RESIDUAL_STORED, SCORE_RANDOM, SCORE_QK, SCORE_ATTN = 0, 1, 2, 3, 4


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a, ctype):
    return None if a is None else a.ctypes.data_as(C.POINTER(ctype))


def lib():
    global _LIB
    if _LIB is None:
        import importlib.util
        spec = importlib.util.spec_from_file_location("_oracle_build", os.path.join(_HERE, "build.py"))
        mod = importlib.util.module_from_spec(spec)
        spec.loader.exec_module(mod)
        # (OVGGT_ORACLE_LIBRARY: another build of the oracle, for the test that plants mistakes in copies of it)
        L = C.CDLL(os.environ.get("OVGGT_ORACLE_LIBRARY") or mod.build())
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.POINTER(OrcConfig)]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_num_rows.argtypes = [C.c_void_p]
        L.orc_num_protected.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.orc_active_anchors.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        L.orc_evicted_total.argtypes = [C.c_void_p]
        L.orc_evicted_total.restype = C.c_int64
        L.orc_attend.argtypes = [C.c_void_p, C.c_int64] + [C.POINTER(C.c_float)] * 3 + [
            C.POINTER(C.c_int32), C.c_int32, C.POINTER(C.c_float)]
        L.orc_compress.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_float), C.c_double,
                                   C.POINTER(C.c_float), C.POINTER(C.c_float), C.POINTER(C.c_int32),
                                   C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
        L.orc_compress_camera.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.c_int32, C.c_int64,
                                          C.POINTER(C.c_float), C.POINTER(C.c_float), C.POINTER(C.c_int32),
                                          C.POINTER(C.c_int32)]
        L.orc_export.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_uint8),
                                 C.POINTER(C.c_float), C.POINTER(C.c_float), C.POINTER(C.c_float)]
        L.orc_residual_norms.argtypes = [C.POINTER(C.c_float), C.c_int32, C.c_int32, C.POINTER(C.c_double)]
        L.orc_qk_scores.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_float), C.c_int32, C.c_int32, C.c_int32,
                                    C.POINTER(C.c_double)]
        L.orc_attention_received.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_float), C.c_int32, C.c_int32,
                                             C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_double)]
        L.orc_smooth.argtypes = [C.POINTER(C.c_double), C.c_int32, C.c_int32, C.c_int32, C.c_double,
                                 C.POINTER(C.c_double)]
        L.orc_diversity.argtypes = [C.POINTER(C.c_float), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                    C.POINTER(C.c_double)]
        L.orc_hybrid.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_uint8),
                                 C.c_int32, C.c_int32, C.c_double, C.POINTER(C.c_float)]
        L.orc_select.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_uint8), C.c_int32, C.c_int32,
                                 C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.orc_top_conf.argtypes = [C.POINTER(C.c_float), C.c_int32, C.c_int32, C.POINTER(C.c_int32)]
        L.orc_attention.argtypes = [C.POINTER(C.c_float)] * 3 + [C.c_int32] * 4 + [
            C.POINTER(C.c_int32), C.c_int32, C.POINTER(C.c_float)]
        L.orc_full_cache_elements.restype = C.c_double
        L.orc_full_cache_elements.argtypes = [C.c_int32, C.c_int64, C.c_int32, C.c_int32, C.c_int32]
        L.orc_set_threads.argtypes = [C.c_int32]
        L.orc_splitmix64.restype = C.c_uint64
        L.orc_splitmix64.argtypes = [C.c_uint64]
        L.orc_random_priority.restype = C.c_float
        L.orc_random_priority.argtypes = [C.c_uint64, C.c_int64, C.c_int64]
        _LIB = L
    return _LIB


def set_threads(n: int) -> None:
    lib().orc_set_threads(int(n))


def get_threads() -> int:
    return int(lib().orc_get_threads())


# ------------------------------------------------------------------ pure pieces

def residual_norms(R: np.ndarray) -> np.ndarray:
    R = _f32(R)
    s = np.empty(R.shape[0], dtype=np.float64)
    lib().orc_residual_norms(_ptr(R, C.c_float), R.shape[0], R.shape[1], _ptr(s, C.c_double))
    return s


def qk_scores(Q: np.ndarray, K: np.ndarray, n_heads: int) -> np.ndarray:
    """Supp. D, query-key criterion: mean scaled logit each of the frame's keys gets from the frame's queries."""
    Q, K = _f32(Q), _f32(K)
    assert Q.shape == K.shape and Q.shape[1] % n_heads == 0
    s = np.empty(Q.shape[0], dtype=np.float64)
    lib().orc_qk_scores(_ptr(Q, C.c_float), _ptr(K, C.c_float), Q.shape[0], n_heads, Q.shape[1] // n_heads,
                        _ptr(s, C.c_double))
    return s


def attention_received(Q: np.ndarray, K: np.ndarray, n_heads: int, first_col: int = 0, n_cols: int = -1) -> np.ndarray:
    """Supp. D, attention-weight criterion: mean over queries and heads of the columns of softmax(Q K^T / sqrt(d))."""
    Q, K = _f32(Q), _f32(K)
    n_cols = K.shape[0] - first_col if n_cols < 0 else n_cols
    s = np.empty(n_cols, dtype=np.float64)
    lib().orc_attention_received(_ptr(Q, C.c_float), _ptr(K, C.c_float), Q.shape[0], K.shape[0], n_heads,
                                 Q.shape[1] // n_heads, first_col, n_cols, _ptr(s, C.c_double))
    return s


def smooth(s: np.ndarray, n_special: int, grid_h: int, grid_w: int, alpha: float) -> np.ndarray:
    s = np.ascontiguousarray(s, dtype=np.float64)
    assert s.shape[0] == n_special + grid_h * grid_w
    out = np.empty_like(s)
    lib().orc_smooth(_ptr(s, C.c_double), n_special, grid_h, grid_w, float(alpha), _ptr(out, C.c_double))
    return out


def diversity(K: np.ndarray, n_heads: int = 1, per_head: bool = False) -> np.ndarray:
    K = _f32(K)
    d = np.empty(K.shape[0], dtype=np.float64)
    lib().orc_diversity(_ptr(K, C.c_float), K.shape[0], K.shape[1], n_heads, int(per_head),
                        _ptr(d, C.c_double))
    return d


def hybrid(d: np.ndarray, s: np.ndarray, flags: np.ndarray, beta: float) -> np.ndarray:
    d = np.ascontiguousarray(d, dtype=np.float64)
    s = np.ascontiguousarray(s, dtype=np.float64)
    flags = np.ascontiguousarray(flags, dtype=np.uint8)
    n, M = d.shape[0], s.shape[0]
    assert flags.shape[0] == n + M
    r = np.empty(n + M, dtype=np.float32)
    lib().orc_hybrid(_ptr(d, C.c_double), _ptr(s, C.c_double), _ptr(flags, C.c_uint8), n, M,
                     float(beta), _ptr(r, C.c_float))
    return r


def select(r: np.ndarray, flags: np.ndarray, budget: int) -> np.ndarray:
    r = _f32(r)
    flags = np.ascontiguousarray(flags, dtype=np.uint8)
    N = r.shape[0]
    out = np.empty(N, dtype=np.int32)
    n_out = C.c_int32(0)
    rc = lib().orc_select(_ptr(r, C.c_float), _ptr(flags, C.c_uint8), N, int(budget),
                          _ptr(out, C.c_int32), C.byref(n_out))
    if rc != 0:
        raise ValueError("protected set exceeds the budget")
    return out[: n_out.value].copy()


def top_conf(conf: np.ndarray, A: int) -> np.ndarray:
    conf = _f32(conf)
    out = np.empty(min(A, conf.shape[0]), dtype=np.int32)
    lib().orc_top_conf(_ptr(conf, C.c_float), conf.shape[0], int(A), _ptr(out, C.c_int32))
    return out


def attention(Q, K, V, n_heads: int, head_dim: int, rows: Optional[Sequence[int]] = None) -> np.ndarray:
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    M, N = Q.shape[0], K.shape[0]
    rows_a = None if rows is None else np.ascontiguousarray(rows, dtype=np.int32)
    n_rows = M if rows_a is None else rows_a.shape[0]
    out = np.empty((n_rows, Q.shape[1]), dtype=np.float32)
    lib().orc_attention(_ptr(Q, C.c_float), _ptr(K, C.c_float), _ptr(V, C.c_float), M, N, n_heads,
                        head_dim, _ptr(rows_a, C.c_int32), n_rows, _ptr(out, C.c_float))
    return out


def splitmix64(x: int) -> int:
    return int(lib().orc_splitmix64(C.c_uint64(x & (2 ** 64 - 1))))


def random_priority(seed: int, frame_id: int, token_id: int) -> float:
    return float(lib().orc_random_priority(C.c_uint64(seed & (2 ** 64 - 1)), int(frame_id), int(token_id)))


def full_cache_elements(L: int, T: int, M: int, n_heads: int, head_dim: int) -> float:
    return float(lib().orc_full_cache_elements(L, T, M, n_heads, head_dim))


# ------------------------------------------------------------------ streaming state

class OracleLayer:
    """The oracle's cache of one layer."""

    def __init__(self, *, n_heads, head_dim, n_special, grid_h, grid_w, budget, anchor_tokens,
                 k_max=3, min_anchor_interval=100, tau=0.2, alpha=0.5, beta=0.5,
                 protect_first_frame=1, score_mode=0, diversity_per_head=0, camera_cache=0, random_seed=0):
        self.cfg = OrcConfig(n_heads, head_dim, n_special, grid_h, grid_w, budget, anchor_tokens,
                             k_max, min_anchor_interval, tau, alpha, beta, protect_first_frame,
                             score_mode, diversity_per_head, camera_cache, random_seed)
        self.M = n_special + grid_h * grid_w
        self.C = n_heads * head_dim
        self._h = lib().orc_create(C.byref(self.cfg))
        if not self._h:
            raise ValueError("invalid oracle config (budget below the protected-set bound?)")

    @classmethod
    def from_stream(cls, cfg, **over) -> "OracleLayer":
        kw = dict(n_heads=cfg.n_heads, head_dim=cfg.head_dim, n_special=cfg.n_special,
                  grid_h=cfg.grid_h, grid_w=cfg.grid_w, budget=cfg.budget,
                  anchor_tokens=cfg.anchor_tokens, k_max=cfg.k_max,
                  min_anchor_interval=cfg.min_anchor_interval, tau=cfg.tau, alpha=cfg.alpha,
                  beta=cfg.beta, protect_first_frame=cfg.protect_first_frame,
                  score_mode=cfg.score_mode, random_seed=cfg.seed)
        kw.update(over)
        return cls(**kw)

    def close(self):
        if self._h:
            lib().orc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def n_rows(self) -> int:
        return int(lib().orc_num_rows(self._h))

    def protected(self):
        a, b = C.c_int32(0), C.c_int32(0)
        lib().orc_num_protected(self._h, C.byref(a), C.byref(b))
        return a.value, b.value

    def anchors(self):
        buf = (C.c_int64 * max(1, self.cfg.k_max + 1))()
        n = lib().orc_active_anchors(self._h, buf)
        return [int(buf[i]) for i in range(n)]

    @property
    def evicted_total(self) -> int:
        return int(lib().orc_evicted_total(self._h))

    def attend(self, frame_id, q, k, v, rows=None, compute=True):
        q, k, v = _f32(q), _f32(k), _f32(v)
        assert q.shape == (self.M, self.C) and k.shape == q.shape and v.shape == q.shape
        rows_a = None if rows is None else np.ascontiguousarray(rows, dtype=np.int32)
        n_rows = self.M if rows_a is None else rows_a.shape[0]
        out = np.empty((n_rows, self.C), dtype=np.float32) if compute else None
        rc = lib().orc_attend(self._h, int(frame_id), _ptr(q, C.c_float), _ptr(k, C.c_float),
                              _ptr(v, C.c_float), _ptr(rows_a, C.c_int32), n_rows, _ptr(out, C.c_float))
        if rc != 0:
            raise RuntimeError(f"orc_attend failed: {rc}")
        return out

    def compress(self, resid, conf=None, rho=float("nan"), score_override=None):
        if resid is None:   # these modes score the frame from what attend() kept
            assert self.cfg.score_mode in (SCORE_QK, SCORE_ATTN)
        else:
            resid = _f32(resid)
            assert resid.shape == (self.M, self.C)
        conf_a = None if conf is None else _f32(conf)
        N = self.n_rows
        ov = None if score_override is None else _f32(score_override)
        if ov is not None:
            assert ov.shape[0] == N
        r = np.empty(N, dtype=np.float32)
        surv = np.empty(N, dtype=np.int32)
        n_s, reg, dem = C.c_int32(0), C.c_int32(0), C.c_int64(-1)
        rc = lib().orc_compress(self._h, _ptr(resid, C.c_float), _ptr(conf_a, C.c_float), float(rho),
                                _ptr(ov, C.c_float), _ptr(r, C.c_float), _ptr(surv, C.c_int32),
                                C.byref(n_s), C.byref(reg), C.byref(dem))
        if rc != 0:
            raise RuntimeError(f"orc_compress failed: {rc}")
        return {"r": r, "survivors": surv[: n_s.value].copy(), "registered": bool(reg.value),
                "demoted_frame": int(dem.value)}

    def compress_camera(self, resid, registered=False, demoted_frame=-1, score_override=None):
        """Supp. C: compress step of the camera head's cache; the anchor decision comes from the aggregator."""
        resid = _f32(resid)
        assert resid.shape == (1, self.C)
        N = self.n_rows
        ov = None if score_override is None else _f32(score_override)
        r = np.empty(N, dtype=np.float32)
        surv = np.empty(N, dtype=np.int32)
        n_s = C.c_int32(0)
        rc = lib().orc_compress_camera(self._h, _ptr(resid, C.c_float), int(bool(registered)), int(demoted_frame),
                                       _ptr(ov, C.c_float), _ptr(r, C.c_float), _ptr(surv, C.c_int32), C.byref(n_s))
        if rc != 0:
            raise RuntimeError(f"orc_compress_camera failed: {rc}")
        return {"r": r, "survivors": surv[: n_s.value].copy()}

    @classmethod
    def camera(cls, *, n_heads, head_dim, budget, k_max=3, beta=0.5, protect_first_frame=1, score_mode=0):
        """The camera head's cache: one token per frame (Supp. C)."""
        return cls(n_heads=n_heads, head_dim=head_dim, n_special=1, grid_h=0, grid_w=0, budget=budget,
                   anchor_tokens=0, k_max=k_max, beta=beta, protect_first_frame=protect_first_frame,
                   score_mode=score_mode, camera_cache=1)

    def export(self, with_kv=True):
        n = self.n_rows
        ids = np.empty(n, dtype=np.int64)
        flags = np.empty(n, dtype=np.uint8)
        stored = np.empty(n, dtype=np.float32)
        k = np.empty((n, self.C), dtype=np.float32) if with_kv else None
        v = np.empty((n, self.C), dtype=np.float32) if with_kv else None
        lib().orc_export(self._h, _ptr(ids, C.c_int64), _ptr(flags, C.c_uint8), _ptr(stored, C.c_float),
                         _ptr(k, C.c_float), _ptr(v, C.c_float))
        return {"ids": ids, "flags": flags, "stored": stored, "k": k, "v": v}
