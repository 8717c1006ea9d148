"""Pins of the CPU oracle to things other than itself: library routines on special
cases, closed forms, brute-force properties on tiny inputs, invariants the paper
states, and the values the paper prints (tests/golden/paper_values.txt)."""
import math
import os

import numpy as np
import pytest
import scipy.ndimage
import scipy.spatial.distance
import torch

from oracle import oracle as orc
from paper_2603_05959_b200 import inputs as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")


def paper_values():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#", 1)[0].strip()
        if line:
            k, v = [x.strip() for x in line.split("=")]
            out[k] = float(v)
    return out


# ------------------------------------------------------------------ attention

def test_attention_matches_library_sdpa_fp64():
    rng = np.random.default_rng(0)
    M, N, H, d = 7, 29, 3, 8          # non-square everywhere so a transposed operand fails
    Q = rng.standard_normal((M, H * d)).astype(np.float32)
    K = rng.standard_normal((N, H * d)).astype(np.float32)
    V = rng.standard_normal((N, H * d)).astype(np.float32)
    got = orc.attention(Q, K, V, H, d)
    q = torch.from_numpy(Q).double().view(M, H, d).transpose(0, 1)
    k = torch.from_numpy(K).double().view(N, H, d).transpose(0, 1)
    v = torch.from_numpy(V).double().view(N, H, d).transpose(0, 1)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v).transpose(0, 1).reshape(M, H * d)
    np.testing.assert_allclose(got, ref.numpy(), rtol=0, atol=2e-7)


def test_attention_closed_forms():
    rng = np.random.default_rng(1)
    M, N, H, d = 4, 11, 2, 4
    Q = rng.standard_normal((M, H * d)).astype(np.float32)
    V = rng.standard_normal((N, H * d)).astype(np.float32)
    # identical keys -> uniform weights -> the mean of V
    K = np.tile(rng.standard_normal((1, H * d)).astype(np.float32), (N, 1))
    np.testing.assert_allclose(orc.attention(Q, K, V, H, d), np.tile(V.mean(0), (M, 1)), atol=1e-6)
    # zero queries -> uniform weights whatever the keys
    K = rng.standard_normal((N, H * d)).astype(np.float32)
    np.testing.assert_allclose(orc.attention(np.zeros_like(Q), K, V, H, d), np.tile(V.mean(0), (M, 1)), atol=1e-6)
    # a single key -> its value row
    np.testing.assert_allclose(orc.attention(Q, K[:1], V[:1], H, d), np.tile(V[:1], (M, 1)), atol=1e-7)
    # one key aligned with the query and huge -> its value row (per head)
    Kbig = K.copy()
    Qa = np.abs(Q[:1]) + 1.0
    Kbig[5] = 50.0 * Qa[0]
    out = orc.attention(Qa, Kbig, V, H, d)
    np.testing.assert_allclose(out[0], V[5], atol=1e-6)


def test_attention_scale_is_inverse_sqrt_head_dim():
    # two keys, one head: weights are softmax([q.k0, q.k1] / sqrt(d)) -> closed form sigmoid
    d = 16
    q = np.zeros((1, d), np.float32); q[0, 0] = 2.0
    K = np.zeros((2, d), np.float32); K[0, 0] = 3.0; K[1, 0] = 1.0
    V = np.zeros((2, d), np.float32); V[0, 0] = 1.0
    w0 = 1.0 / (1.0 + math.exp(-(2.0 * 3.0 - 2.0 * 1.0) / math.sqrt(d)))
    out = orc.attention(q, K, V, 1, d)
    assert abs(out[0, 0] - w0) < 1e-7


def test_attention_permutation_and_row_subset():
    rng = np.random.default_rng(2)
    M, N, H, d = 6, 17, 2, 8
    Q, K, V = (rng.standard_normal(s).astype(np.float32) for s in ((M, H * d), (N, H * d), (N, H * d)))
    full = orc.attention(Q, K, V, H, d)
    perm = rng.permutation(N)
    np.testing.assert_allclose(orc.attention(Q, K[perm], V[perm], H, d), full, atol=1e-6)
    rows = [4, 1]
    np.testing.assert_array_equal(orc.attention(Q, K, V, H, d, rows=rows), full[rows])
    # heads are independent: changing head 1's keys leaves head 0's output alone
    K2 = K.copy(); K2[:, d:] += 1.0
    np.testing.assert_array_equal(orc.attention(Q, K2, V, H, d)[:, :d], full[:, :d])


# ------------------------------------------------------------------ Eq. 5 / Eq. 6

def test_residual_norm_closed_forms():
    R = np.zeros((3, 8), np.float32)
    R[0, 5] = -3.0                     # one-hot row -> |entry|
    R[1, :] = 2.0                      # constant row -> 2 sqrt(C)
    R[2, 0], R[2, 1] = 3.0, 4.0        # 3-4-5
    np.testing.assert_allclose(orc.residual_norms(R), [3.0, 2.0 * math.sqrt(8), 5.0], rtol=1e-15)
    rng = np.random.default_rng(3)
    X = rng.standard_normal((5, 33)).astype(np.float32)
    np.testing.assert_allclose(orc.residual_norms(X), np.linalg.norm(X.astype(np.float64), axis=1), rtol=1e-14)
    np.testing.assert_allclose(orc.residual_norms(4.0 * X), 4.0 * orc.residual_norms(X), rtol=1e-14)


def test_smoothing_special_cases():
    rng = np.random.default_rng(4)
    ns, gh, gw = 5, 6, 9
    s = rng.random(ns + gh * gw)
    # alpha = 0 is the identity
    np.testing.assert_array_equal(orc.smooth(s, ns, gh, gw, 0.0), s)
    # a constant map is a fixed point under the replicate border, and aux tokens are untouched
    c = np.concatenate([s[:ns], np.full(gh * gw, 2.5)])
    out = orc.smooth(c, ns, gh, gw, 0.7)
    np.testing.assert_array_equal(out[:ns], s[:ns])
    np.testing.assert_allclose(out[ns:], 2.5, rtol=1e-15)
    # alpha = 1 equals the library's separable Gaussian filter (sigma 1, radius 1, nearest border)
    lib = scipy.ndimage.gaussian_filter(s[ns:].reshape(gh, gw), sigma=1.0, truncate=1.0, mode="nearest")
    np.testing.assert_allclose(orc.smooth(s, ns, gh, gw, 1.0)[ns:].reshape(gh, gw), lib, rtol=1e-13)
    # general alpha is the blend of the two
    a = 0.3
    np.testing.assert_allclose(orc.smooth(s, ns, gh, gw, a)[ns:].reshape(gh, gw),
                               a * lib + (1 - a) * s[ns:].reshape(gh, gw), rtol=1e-13)


def test_smoothing_impulse_gives_kernel_and_preserves_mass():
    ns, gh, gw = 2, 7, 5               # non-square: a transposed map would fail
    s = np.zeros(ns + gh * gw); s[ns + 3 * gw + 2] = 1.0
    out = orc.smooth(s, ns, gh, gw, 1.0)[ns:].reshape(gh, gw)
    z = 1.0 + 4 * math.exp(-0.5) + 4 * math.exp(-1.0)
    assert abs(out[3, 2] - 1.0 / z) < 1e-15
    assert abs(out[2, 2] - math.exp(-0.5) / z) < 1e-15 and abs(out[3, 1] - math.exp(-0.5) / z) < 1e-15
    assert abs(out[2, 1] - math.exp(-1.0) / z) < 1e-15
    assert abs(out.sum() - 1.0) < 1e-14 and out[0, 0] == 0.0


# ------------------------------------------------------------------ diversity / Eq. 7

def test_diversity_closed_forms():
    e = np.eye(4, dtype=np.float32)
    # two orthonormal keys: centroid (a+b)/2, cos = 1/sqrt(2)
    d = orc.diversity(np.stack([e[0], e[1]]))
    np.testing.assert_allclose(d, 1 - 1 / math.sqrt(2), rtol=1e-15)
    # identical keys: d = 0; positive scaling of a key does not change its d
    K = np.stack([2 * e[0] + e[1], 6 * e[0] + 3 * e[1]])
    np.testing.assert_allclose(orc.diversity(K), 0.0, atol=1e-15)
    # opposite of the centroid direction: d = 2
    K = np.stack([e[0], e[0], e[0], -e[0]])
    np.testing.assert_allclose(orc.diversity(K), [0, 0, 0, 2], atol=1e-15)
    # a zero key has cosine 0 by convention
    K = np.stack([e[0], np.zeros(4, np.float32)])
    np.testing.assert_allclose(orc.diversity(K), [0, 1], atol=1e-15)


def test_diversity_matches_library_cosine_distance():
    rng = np.random.default_rng(5)
    K = rng.standard_normal((13, 24)).astype(np.float32)
    kbar = K.astype(np.float64).mean(0)
    ref = [scipy.spatial.distance.cosine(k.astype(np.float64), kbar) for k in K]
    np.testing.assert_allclose(orc.diversity(K), ref, rtol=1e-12)
    # per-head variant: mean over heads of the per-head cosine distance
    ref_h = [np.mean([scipy.spatial.distance.cosine(k[h * 8:(h + 1) * 8].astype(np.float64),
                                                    kbar[h * 8:(h + 1) * 8]) for h in range(3)]) for k in K]
    np.testing.assert_allclose(orc.diversity(K, n_heads=3, per_head=True), ref_h, rtol=1e-12)


def test_hybrid_normalisation_properties():
    rng = np.random.default_rng(6)
    n, M, beta = 40, 12, 0.3
    d, s = rng.random(n) * 2, rng.random(M) * 50 + 3
    flags = np.zeros(n + M, np.uint8)
    flags[[0, 7, n + 2]] = [1, 2, 2]
    d[0], d[7], s[2] = 1e9, -1e9, 1e9        # protected rows must not enter the min / max
    r = orc.hybrid(d, s, flags, beta)
    ev_h = np.flatnonzero(flags[:n] == 0); ev_n = n + np.flatnonzero(flags[n:] == 0)
    assert np.all(np.isinf(r[flags != 0])) and np.all(r[flags != 0] > 0)
    assert r[ev_h].min() == 0.0 and r[ev_h].max() == np.float32(1 - beta)
    assert r[ev_n].min() == 0.0 and r[ev_n].max() == np.float32(beta)
    # where the extremes sit, and the order inside each group
    assert ev_h[np.argmax(r[ev_h])] == ev_h[np.argmax(d[ev_h])]
    assert np.array_equal(np.argsort(r[ev_n], kind="stable"), np.argsort(s[ev_n - n], kind="stable"))
    # affine invariance of min-max
    r2 = orc.hybrid(3 * d + 5, 0.1 * s - 2, flags, beta)
    np.testing.assert_allclose(r2[flags == 0], r[flags == 0], rtol=0, atol=1e-7)
    # an explicit value: the mid-point of a 3-member group
    r3 = orc.hybrid(np.array([1.0, 2.0, 3.0]), np.array([4.0]), np.zeros(4, np.uint8), 0.25)
    np.testing.assert_allclose(r3, [0.0, 0.375, 0.75, 0.0], atol=1e-7)
    # degenerate weights and ranges
    assert np.all(orc.hybrid(d, s, flags, 1.0)[ev_h] == 0.0)
    assert np.all(orc.hybrid(d, s, flags, 0.0)[ev_n] == 0.0)
    assert np.all(orc.hybrid(np.full(n, 0.7), s, flags, beta)[ev_h] == 0.0)


# ------------------------------------------------------------------ Eq. 8

def brute_force_keep(r, flags, B):
    """Definition of Eq. 8 with the tie rule, via numpy's stable argsort (a library sort)."""
    N = len(r)
    if N <= B:
        return np.arange(N)
    key = np.where(np.isnan(r), -np.inf, r).astype(np.float32)
    ev = np.flatnonzero(flags == 0)
    order = ev[np.argsort(-key[ev], kind="stable")]
    keep = np.concatenate([np.flatnonzero(flags != 0), order[: B - np.count_nonzero(flags)]])
    return np.sort(keep)


@pytest.mark.parametrize("seed", range(6))
def test_select_matches_brute_force_with_heavy_ties(seed):
    rng = np.random.default_rng(100 + seed)
    N = int(rng.integers(5, 60))
    levels = rng.choice([2, 3, 50])
    r = rng.integers(0, levels, N).astype(np.float32) / np.float32(levels)
    if seed % 2:
        r[rng.integers(0, N, 3)] = [np.nan, -np.inf, np.inf]
        r[rng.integers(0, N)] = -0.0
    flags = (rng.random(N) < 0.2).astype(np.uint8) * rng.integers(1, 3, N).astype(np.uint8)
    P = int(np.count_nonzero(flags))
    for B in sorted({P, P + 1, (P + N) // 2, N - 1, N, N + 3}):
        got = orc.select(r, flags, B)
        np.testing.assert_array_equal(got, brute_force_keep(r, flags, B))
        assert len(got) == min(N, B)
        assert set(np.flatnonzero(flags)).issubset(set(got.tolist()))
        # pairwise statement of the rule: no dropped evictable row outranks a kept one
        key = np.where(np.isnan(r), -np.inf, r)
        kept = set(got.tolist())
        for i in range(N):
            for j in range(N):
                if flags[i] == 0 and flags[j] == 0 and i in kept and j not in kept:
                    assert key[i] > key[j] or (key[i] == key[j] and i < j)


def test_select_explicit_tie_case():
    r = np.array([0.5, 0.5, 0.5, 0.9, 0.5, 0.1], np.float32)
    flags = np.array([0, 0, 0, 0, 0, 1], np.uint8)
    np.testing.assert_array_equal(orc.select(r, flags, 4), [0, 1, 3, 5])   # 5 protected, 3 best, ties 0 and 1
    np.testing.assert_array_equal(orc.select(r, flags, 1), [5])            # budget = |P|: all evictable dropped
    with pytest.raises(ValueError):
        orc.select(r, np.ones(6, np.uint8), 3)
    np.testing.assert_array_equal(orc.select(np.array([0.0, -0.0, 0.0], np.float32), np.zeros(3, np.uint8), 2), [0, 1])


def test_top_conf():
    conf = np.array([0.3, 0.9, 0.9, np.nan, 0.1, 0.9], np.float32)
    np.testing.assert_array_equal(orc.top_conf(conf, 2), [1, 2])
    np.testing.assert_array_equal(orc.top_conf(conf, 4), [0, 1, 2, 5])
    np.testing.assert_array_equal(orc.top_conf(conf, 6), np.arange(6))


# ------------------------------------------------------------------ the paper's printed values

def test_paper_token_count_and_memory_model():
    pv = paper_values()
    M = 1 + 4 + (518 // 14) * (392 // 14)
    assert M == pv["tokens_per_frame_518x392_p14"]
    elems = orc.full_cache_elements(int(pv["n_layers"]), 100, M, 16, 64)
    assert elems == 2 * 24 * 100 * 1041 * 16 * 64
    gb = elems * 2 / 1e9                                  # 2-byte elements
    assert abs(gb - pv["full_cache_gb_at_100_frames"]) < 0.5
    assert 100 * M > pv["full_cache_tokens_per_layer_100_frames_min"]
    # default budget of 200K tokens over all layers, 2 * C * 2 bytes per token: doubling adds about 1 GB
    extra = pv["default_budget_tokens"] * 2 * 1024 * 2 / 1e9
    assert abs(extra - pv["budget_400k_extra_gb"]) < 0.25
    # Eq. 9 at the paper's defaults: 1041 + 3 * ceil(0.05 * 1036) = 1197
    assert M + int(pv["k_max"]) * math.ceil(pv["eta"] * (M - 5)) == 1197


# ------------------------------------------------------------------ anchors and stream invariants

def _tiny_layer(**over):
    kw = dict(n_heads=2, head_dim=4, n_special=2, grid_h=3, grid_w=4, budget=60, anchor_tokens=3,
              k_max=2, min_anchor_interval=3, tau=0.2)
    kw.update(over)
    return orc.OracleLayer(**kw)


def _step(layer, t, rng, rho, conf=None, **kw):
    M, C = layer.M, layer.C
    q, k, v, r = (rng.standard_normal((M, C)).astype(np.float32) for _ in range(4))
    layer.attend(t, q, k, v, compute=False)
    return layer.compress(r, conf if conf is not None else rng.random(M - 2).astype(np.float32), rho, **kw)


def test_anchor_fifo_on_handwritten_schedule():
    layer = _tiny_layer()
    rng = np.random.default_rng(7)
    M = layer.M
    #        t:  0    1    2    3    4    5    6    7    8    9   10   11   12
    rhos = [0.0, 0.0, 0.0, 0.5, 0.1, 0.0, 0.0, 0.0, 0.9, 0.0, 0.0, 0.0, 0.1]
    # frame 0 is the initial anchor (never "registered"); interval 3 -> earliest t = 3, where rho = 0.5 fails;
    # t = 4 registers; next allowed t >= 7 -> 7 registers; 8 fails on rho; 10 registers (t - 7 = 3) and,
    # with K_max = 2, releases anchor 4; 12 is too early (12 - 10 < 3).
    expect_reg = {4, 7, 10}
    expect_anchors = {4: [4], 7: [4, 7], 10: [7, 10], 12: [7, 10]}
    for t, rho in enumerate(rhos):
        conf = np.zeros(M - 2, np.float32)
        conf[[1, 5, 9]] = [3.0, 2.0, 1.0]
        out = _step(layer, t, rng, rho, conf)
        assert out["registered"] == (t in expect_reg)
        assert out["demoted_frame"] == (4 if t == 10 else -1)
        if t in expect_anchors:
            assert layer.anchors() == expect_anchors[t]
        ex = layer.export(with_kv=False)
        hist = ex["ids"][ex["flags"] == 2]
        want = sorted(a * M + 2 + p for a in layer.anchors() for p in (1, 5, 9))
        assert sorted(hist.tolist()) == want
    # NaN coverage never registers; a missing confidence map neither
    layer2 = _tiny_layer()
    for t in range(6):
        M2, C2 = layer2.M, layer2.C
        x = np.ones((M2, C2), np.float32)
        layer2.attend(t, x, x, x, compute=False)
        out = layer2.compress(x, None if t % 2 else np.ones(M2 - 2, np.float32), float("nan") if t % 2 == 0 else 0.0)
        assert not out["registered"]


@pytest.mark.parametrize("tau", [0.2, 0.9])
def test_stream_invariants_budget_anchors_first_frame(tau):
    cfg = gen.config_tiny().replace(tau=tau)
    layer = orc.OracleLayer.from_stream(cfg)
    M, B = cfg.tokens_per_frame, cfg.budget
    bound = M + cfg.k_max * cfg.anchor_tokens
    evicted = 0
    for t in range(cfg.n_frames):
        fi = gen.frame_inputs(cfg, t)
        n_before = layer.n_rows
        layer.attend(t, fi.q, fi.k, fi.v, compute=False)
        out = layer.compress(fi.resid, fi.conf, fi.rho)
        N = n_before + M
        assert layer.n_rows == min(N, B)                       # Eq. 8 / the budget invariant
        evicted += N - layer.n_rows
        ex = layer.export(with_kv=False)
        assert np.all(np.diff(ex["ids"]) > 0)                  # order-preserving compaction
        assert np.array_equal(ex["ids"][:M], np.arange(M))     # first-frame tokens stay for good
        assert np.all(ex["flags"][:M] == 1)
        n_init, n_hist = layer.protected()
        assert n_init == M and n_init + n_hist <= bound        # Eq. 9
        assert n_hist == cfg.anchor_tokens * len(layer.anchors())
        assert len(layer.anchors()) <= cfg.k_max
        assert np.all(np.isinf(out["r"][:M]))
    assert layer.evicted_total == evicted and evicted > 0
    assert len(layer.anchors()) >= 1
    if tau > 0.5:
        assert len(layer.anchors()) == cfg.k_max               # frequent triggers exercise the FIFO


def test_compress_layout_is_gather_of_inputs():
    """Rows that survive carry exactly the K/V/ids they were appended with."""
    cfg = gen.config_tiny().replace(budget=150, anchor_tokens=4)
    layer = orc.OracleLayer.from_stream(cfg)
    M = cfg.tokens_per_frame
    seen_k, seen_v = {}, {}
    for t in range(5):
        fi = gen.frame_inputs(cfg, t)
        for j in range(M):
            seen_k[t * M + j], seen_v[t * M + j] = fi.k[j], fi.v[j]
        layer.attend(t, fi.q, fi.k, fi.v, compute=False)
        pre_ids = np.concatenate([layer.export(with_kv=False)["ids"]])
        out = layer.compress(fi.resid, fi.conf, fi.rho)
        ex = layer.export()
        np.testing.assert_array_equal(ex["ids"], pre_ids[out["survivors"]])
        for row, tid in enumerate(ex["ids"]):
            assert np.array_equal(ex["k"][row], seen_k[int(tid)]) and np.array_equal(ex["v"][row], seen_v[int(tid)])


def test_score_override_and_stored_mode():
    cfg = gen.config_tiny().replace(budget=100, anchor_tokens=0)
    a = orc.OracleLayer.from_stream(cfg)
    b = orc.OracleLayer.from_stream(cfg, score_mode=1)
    M = cfg.tokens_per_frame
    for t in range(3):
        fi = gen.frame_inputs(cfg, t)
        a.attend(t, fi.q, fi.k, fi.v, compute=False)
        b.attend(t, fi.q, fi.k, fi.v, compute=False)
        N = a.n_rows
        ov = np.linspace(1.0, 0.0, N).astype(np.float32)       # prefer old rows: the newest are evicted
        oa = a.compress(fi.resid, fi.conf, fi.rho, score_override=ov)
        ob = b.compress(fi.resid, fi.conf, fi.rho)
        np.testing.assert_array_equal(oa["survivors"], np.arange(min(N, cfg.budget)))
        # stored-residual mode ranks by the smoothed norm each row had when new
        s = orc.smooth(orc.residual_norms(fi.resid), cfg.n_special, cfg.grid_h, cfg.grid_w, cfg.alpha)
        if t > 0:
            np.testing.assert_array_equal(ob["r"][-M:], s.astype(np.float32))
    ex = b.export(with_kv=False)
    assert np.all(ex["stored"] > 0)


def test_stored_scores_travel_with_their_rows_through_every_compaction():
    """Stored-residual reading of the score (Sec. 3.2, Activation Value Rating + smoothing): a cached row ranks by
    the smoothed norm it received in the frame that brought it in.  That value has to move with the row every time
    the cache is compacted.  Expected values are rebuilt here per token id from each frame's own residual (numpy
    norm, scipy Gaussian for the interior of the map) and compared, after several evictions, with what the oracle
    exports and with the priorities it ranks the historical rows by."""
    cfg = gen.config_tiny().replace(score_mode=gen.SCORE_RESIDUAL_STORED, budget=150, anchor_tokens=4,
                                    min_anchor_interval=3, tau=0.9)
    layer = orc.OracleLayer.from_stream(cfg)
    M, ns, gh, gw = cfg.tokens_per_frame, cfg.n_special, cfg.grid_h, cfg.grid_w
    expected = {}                                             # token id -> fp32 score it was given when new
    evictions = 0
    for t in range(9):
        fi = gen.frame_inputs(cfg, t)
        s = np.linalg.norm(fi.resid.astype(np.float64), axis=1)
        sm = orc.smooth(s, ns, gh, gw, cfg.alpha)
        # the interior of the patch map against a library Gaussian (3x3, sigma 1 == truncate 1)
        lib_map = scipy.ndimage.gaussian_filter(s[ns:].reshape(gh, gw), sigma=1.0, truncate=1.0, mode="nearest")
        np.testing.assert_allclose(sm[ns:].reshape(gh, gw), cfg.alpha * lib_map + (1 - cfg.alpha) * s[ns:].reshape(gh, gw),
                                   rtol=1e-12)
        for j in range(M):
            expected[t * M + j] = np.float32(sm[j])
        layer.attend(t, fi.q, fi.k, fi.v, compute=False)
        pre = layer.export(with_kv=False)                     # pre-compaction ids and flags (new rows appended)
        out = layer.compress(fi.resid, fi.conf, fi.rho)
        n = len(pre["ids"]) - M
        evictions += len(pre["ids"]) - len(out["survivors"]) > 0
        # historical evictable rows rank by the value they were given when new, whatever moved in between
        hist = [i for i in range(n) if np.isfinite(out["r"][i])]
        assert all(out["r"][i] == expected[int(pre["ids"][i])] for i in hist), t
        if t > 2:
            assert len(hist) > 0
        # new rows rank by this frame's smoothed norms
        newfin = [j for j in range(M) if np.isfinite(out["r"][n + j])]
        assert all(out["r"][n + j] == np.float32(sm[j]) for j in newfin)
        # and every survivor carries its own value, not a neighbour's
        ex = layer.export(with_kv=False)
        want = np.array([expected[int(i)] for i in ex["ids"]], dtype=np.float32)
        np.testing.assert_array_equal(ex["stored"], want, err_msg=f"frame {t}")
    assert evictions >= 5                                     # the carry was exercised repeatedly
    # rows of several different frames are still present, so a carry error could not hide behind a single frame
    assert len({int(i) // M for i in layer.export(with_kv=False)["ids"]}) >= 3


# ------------------------------------------------------------------ Supp. A: the random-eviction baseline

def test_splitmix64_reference_outputs_and_priority_range():
    """The generator behind the random-eviction baseline against the published reference outputs of SplitMix64
    (state 0: the first three outputs), and the priority against the formula written out with Python integers."""
    golden = 0x9E3779B97F4A7C15
    assert orc.splitmix64(0) == 0xE220A8397B1DCDAF
    assert orc.splitmix64(golden) == 0x6E789E6AA1B965F4
    assert orc.splitmix64(2 * golden) == 0x06C45D188009454F

    def mix(x):
        m = 2 ** 64 - 1
        z = (x + golden) & m
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & m
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & m
        return z ^ (z >> 31)

    us = []
    for seed, t, tok in [(0, 0, 0), (20260305, 7, 483), (2 ** 63 + 5, 9999, 13_739_999), (1, 2, 3)]:
        want = (mix((mix(seed ^ t) + tok) & (2 ** 64 - 1)) >> 40) / 2.0 ** 24
        got = orc.random_priority(seed, t, tok)
        assert got == want and 0.0 <= got < 1.0
        us.append(got)
    assert len(set(us)) == 4
    u = np.array([orc.random_priority(5, 3, i) for i in range(20000)])
    assert abs(u.mean() - 0.5) < 0.01 and abs(np.mean(u < 0.1) - 0.1) < 0.01      # uniform, roughly


def test_random_eviction_mode_keeps_a_uniform_subset_and_every_protected_row():
    cfg = gen.config_tiny().replace(score_mode=gen.SCORE_RANDOM, budget=150, anchor_tokens=4, min_anchor_interval=3,
                                    tau=0.9, n_frames=40)
    layer = orc.OracleLayer.from_stream(cfg)
    M = cfg.tokens_per_frame
    evicted_pos = []
    for t in range(cfg.n_frames):
        fi = gen.frame_inputs(cfg, t)
        layer.attend(t, fi.q, fi.k, fi.v, compute=False)
        pre = layer.export(with_kv=False)
        out = layer.compress(fi.resid, fi.conf, fi.rho)
        fin = np.isfinite(out["r"])
        want = np.array([orc.random_priority(cfg.seed, t, int(i)) for i in pre["ids"]], dtype=np.float32)
        np.testing.assert_array_equal(out["r"][fin], want[fin])
        # Eq. 8 on those priorities, by brute force
        N = len(pre["ids"])
        if N > cfg.budget:
            prot = np.flatnonzero(~fin)
            order = sorted(np.flatnonzero(fin), key=lambda i: (-out["r"][i], i))[: cfg.budget - len(prot)]
            np.testing.assert_array_equal(out["survivors"], np.sort(np.concatenate([prot, order])))
            gone = np.setdiff1d(np.arange(N), out["survivors"])
            evicted_pos += (gone / N).tolist()
        ex = layer.export(with_kv=False)
        assert np.array_equal(ex["ids"][:M], np.arange(M))                       # the first frame stays
    # evictions fall all over the buffer, old rows and new rows alike (a score-based rule would not do that)
    hist = np.histogram(evicted_pos, bins=4, range=(0, 1))[0] / len(evicted_pos)
    assert len(evicted_pos) > 1500 and hist[1:].min() > 0.15


# ------------------------------------------------------------------ Supp. D: the query-key criterion

def test_qk_scores_are_the_mean_scaled_logits_a_key_receives():
    """Against the library's batched matmul: the logits softmax would see, averaged over queries and heads; and the
    closed form through the mean query.  M, H, d all differ and Q is not K, so a transposed operand, a sum over the
    wrong axis or a missing 1/sqrt(d) fails."""
    rng = np.random.default_rng(11)
    M, H, d = 13, 3, 8
    Q = rng.standard_normal((M, H * d)).astype(np.float32) + 0.3
    K = rng.standard_normal((M, H * d)).astype(np.float32) - 0.2
    got = orc.qk_scores(Q, K, H)
    q = torch.from_numpy(Q).double().view(M, H, d).transpose(0, 1)      # [H, M, d]
    k = torch.from_numpy(K).double().view(M, H, d).transpose(0, 1)
    logits = torch.matmul(q, k.transpose(1, 2)) / math.sqrt(d)          # [H, i, j]
    want = logits.mean(dim=(0, 1)).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)
    qbar = Q.astype(np.float64).mean(axis=0)                            # one C-vector
    np.testing.assert_allclose(got, K.astype(np.float64) @ qbar / (H * math.sqrt(d)), rtol=1e-12, atol=1e-13)
    assert np.abs(got - orc.qk_scores(K, Q, H)).max() > 1e-3             # queries and keys are not interchangeable
    # a key that is the zero vector receives logit 0 from everyone; scaling the keys scales the scores
    K2 = K.copy(); K2[4] = 0.0
    assert orc.qk_scores(Q, K2, H)[4] == 0.0
    np.testing.assert_allclose(orc.qk_scores(Q, 2.0 * K, H), 2.0 * got, rtol=1e-12)


def test_qk_mode_replaces_only_the_current_frame_criterion():
    """The stream in query-key mode: the new rows' priorities are beta x min-max of the smoothed query-key scores
    (recomputed here with numpy and scipy), the cached rows' priorities equal those of the hybrid mode on the same
    cache, and the residual plays no part."""
    base = gen.config_tiny().replace(anchor_tokens=0, n_frames=8, budget=10_000)      # nothing is evicted: same caches
    cfg = base.replace(score_mode=gen.SCORE_QK)
    qk, hy = orc.OracleLayer.from_stream(cfg), orc.OracleLayer.from_stream(base)
    M, H, d = cfg.tokens_per_frame, cfg.n_heads, cfg.head_dim
    for t in range(cfg.n_frames):
        fi = gen.frame_inputs(cfg, t)
        qk.attend(t, fi.q, fi.k, fi.v, compute=False)
        hy.attend(t, fi.q, fi.k, fi.v, compute=False)
        out = qk.compress(None, fi.conf, fi.rho)
        ref = hy.compress(fi.resid, fi.conf, fi.rho)
        n = len(out["r"]) - M
        if t == 0:
            assert np.all(np.isinf(out["r"]))                                          # first frame: protected
            continue
        np.testing.assert_array_equal(out["r"][:n], ref["r"][:n])                      # (1 - beta) x diversity part
        s = (fi.k.astype(np.float64) @ fi.q.astype(np.float64).mean(axis=0)) / (H * math.sqrt(d))
        grid = s[cfg.n_special:].reshape(cfg.grid_h, cfg.grid_w)
        g = np.exp(-0.5 * np.array([[2, 1, 2], [1, 0, 1], [2, 1, 2]], dtype=np.float64))
        sm = s.copy()
        sm[cfg.n_special:] = ((1 - cfg.alpha) * grid + cfg.alpha * scipy.ndimage.correlate(
            grid, g / g.sum(), mode="nearest")).ravel()
        want = cfg.beta * (sm - sm.min()) / (sm.max() - sm.min())
        np.testing.assert_allclose(out["r"][n:], want, rtol=0, atol=2e-6)
        assert np.abs(out["r"][n:] - ref["r"][n:]).max() > 0.05                        # not the residual criterion
        np.testing.assert_allclose(qk.export(with_kv=False)["stored"][n:], sm, rtol=1e-6)


def test_attention_received_is_the_column_mean_of_the_librarys_softmax():
    """The attention-weight criterion (Supp. D) against torch's softmax of the library matmul's logits: the mean over
    heads and queries of each key's column.  M, N, H, d all differ.  Over all columns the means add up to 1 (every row
    of P does); with all-zero queries every key receives exactly 1 / N."""
    rng = np.random.default_rng(21)
    M, N, H, d = 5, 17, 3, 8
    Q = rng.standard_normal((M, H * d)).astype(np.float32)
    K = rng.standard_normal((N, H * d)).astype(np.float32) * 1.5
    q = torch.from_numpy(Q).double().view(M, H, d).transpose(0, 1)
    k = torch.from_numpy(K).double().view(N, H, d).transpose(0, 1)
    P = torch.softmax(torch.matmul(q, k.transpose(1, 2)) / math.sqrt(d), dim=-1)      # [H, M, N]
    want = P.mean(dim=(0, 1)).numpy()
    got = orc.attention_received(Q, K, H)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)
    assert abs(got.sum() - 1.0) < 1e-12
    np.testing.assert_allclose(orc.attention_received(Q, K, H, first_col=N - 4, n_cols=4), want[N - 4:], rtol=1e-12)
    np.testing.assert_allclose(orc.attention_received(np.zeros_like(Q), K, H), np.full(N, 1.0 / N), rtol=1e-14)
    # a key every query points at collects (nearly) all the attention
    K2 = K.copy(); K2[3] = 0.0
    Q2 = np.tile(np.ones((1, H * d), dtype=np.float32) * 3.0, (M, 1)); K2[3] = 3.0
    assert orc.attention_received(Q2, K2, H)[3] > 0.99


def test_attention_weight_mode_scores_the_frame_by_the_attention_it_receives():
    """The stream in attention-weight mode: the new rows' priorities are beta x min-max of the smoothed attention the
    frame's tokens receive in the frame's own attention over [cache + frame] (recomputed here with numpy), the cached
    rows' priorities equal the hybrid mode's, the residual plays no part."""
    base = gen.config_tiny().replace(anchor_tokens=0, n_frames=6, budget=10_000)
    cfg = base.replace(score_mode=gen.SCORE_ATTN)
    aw, hy = orc.OracleLayer.from_stream(cfg), orc.OracleLayer.from_stream(base)
    M, H, d = cfg.tokens_per_frame, cfg.n_heads, cfg.head_dim
    for t in range(cfg.n_frames):
        fi = gen.frame_inputs(cfg, t)
        aw.attend(t, fi.q, fi.k, fi.v, compute=False)
        hy.attend(t, fi.q, fi.k, fi.v, compute=False)
        keys = aw.export()["k"].astype(np.float64)                                     # cache + frame, N rows
        out = aw.compress(None, fi.conf, fi.rho)
        ref = hy.compress(fi.resid, fi.conf, fi.rho)
        n = len(out["r"]) - M
        if t == 0:
            continue
        np.testing.assert_array_equal(out["r"][:n], ref["r"][:n])
        qh = fi.q.astype(np.float64).reshape(M, H, d).transpose(1, 0, 2)
        kh = keys.reshape(-1, H, d).transpose(1, 0, 2)
        logits = qh @ kh.transpose(0, 2, 1) / math.sqrt(d)
        P = np.exp(logits - logits.max(axis=-1, keepdims=True))
        P /= P.sum(axis=-1, keepdims=True)
        s = P.mean(axis=(0, 1))[n:]
        grid = s[cfg.n_special:].reshape(cfg.grid_h, cfg.grid_w)
        g = np.exp(-0.5 * np.array([[2, 1, 2], [1, 0, 1], [2, 1, 2]], dtype=np.float64))
        sm = s.copy()
        sm[cfg.n_special:] = ((1 - cfg.alpha) * grid + cfg.alpha * scipy.ndimage.correlate(
            grid, g / g.sum(), mode="nearest")).ravel()
        want = cfg.beta * (sm - sm.min()) / (sm.max() - sm.min())
        np.testing.assert_allclose(out["r"][n:], want, rtol=0, atol=2e-6)
        assert np.abs(out["r"][n:] - ref["r"][n:]).max() > 0.05


# ------------------------------------------------------------------ Supp. C: the camera head's cache

def _camera_token(cfg, t, tag):
    """One seeded row of `cfg.dim` values for frame t (the camera token's q, k, v or residual)."""
    rng = np.random.Generator(np.random.Philox(key=[np.uint64(cfg.seed + 77), np.uint64((t << 8) | tag)]))
    return gen.round_to_dtype(rng.standard_normal((1, cfg.dim), dtype=np.float32) * (1.0 + 0.1 * tag), cfg.dtype)


def test_camera_cache_follows_the_aggregators_anchor_schedule():
    """One token per frame under the same scoring and protection (Supp. C).  The aggregator oracle runs a stream with
    frequent anchor turnover; its decision of each frame (registered, demoted frame) drives the camera cache.  The
    camera cache's protected tokens must be exactly the first frame and the aggregator's active anchors after every
    frame, never be evicted while active, and the cache must hold min(t + 1, B_cam) tokens."""
    cfg = gen.config_tiny().replace(tau=0.95, min_anchor_interval=2, k_max=2, n_frames=30)
    agg = orc.OracleLayer.from_stream(cfg)
    cam = orc.OracleLayer.camera(n_heads=cfg.n_heads, head_dim=cfg.head_dim, budget=7, k_max=cfg.k_max)
    demotions = 0
    for t in range(cfg.n_frames):
        fi = gen.frame_inputs(cfg, t)
        agg.attend(t, fi.q, fi.k, fi.v, compute=False)
        dec = agg.compress(fi.resid, fi.conf, fi.rho)
        demotions += dec["demoted_frame"] >= 0
        cam.attend(t, _camera_token(cfg, t, 1), _camera_token(cfg, t, 2), _camera_token(cfg, t, 3), compute=False)
        cam.compress_camera(_camera_token(cfg, t, 4), dec["registered"], dec["demoted_frame"])
        ex = cam.export(with_kv=False)
        assert len(ex["ids"]) == min(t + 1, 7) and np.all(np.diff(ex["ids"]) > 0)
        assert ex["ids"][0] == 0 and ex["flags"][0] == 1                       # the first frame's token, for good
        assert sorted(ex["ids"][ex["flags"] == 2].tolist()) == agg.anchors()   # the same anchors, token for token
        assert cam.anchors() == agg.anchors()
    assert demotions >= 3 and len(agg.anchors()) == 2


def test_camera_cache_scores_closed_forms():
    """No smoothing: the stored score is the raw residual norm.  The lone new token ranks at beta exactly; cached
    tokens at (1 - beta) x the min-max of their cosine distances to the centroid key (library cosine)."""
    C, H = 128, 2
    cam = orc.OracleLayer.camera(n_heads=H, head_dim=64, budget=5, beta=0.3, protect_first_frame=0)
    rng = np.random.default_rng(8)
    keys, norms = [], []
    for t in range(9):
        q, k, v, r = (rng.standard_normal((1, C)).astype(np.float32) for _ in range(4))
        keys.append(k[0]); norms.append(np.float32(np.linalg.norm(r.astype(np.float64))))
        cam.attend(t, q, k, v, compute=False)
        pre = cam.export(with_kv=False)
        out = cam.compress_camera(r)
        n = len(pre["ids"]) - 1
        assert out["r"][n] == np.float32(0.3)                                   # beta x 1
        if n >= 2:
            K = np.stack([keys[int(i)] for i in pre["ids"][:n]]).astype(np.float64)
            d = np.array([scipy.spatial.distance.cosine(k_, K.mean(0)) for k_ in K])
            want = 0.7 * (d - d.min()) / (d.max() - d.min())
            np.testing.assert_allclose(out["r"][:n], want, rtol=0, atol=1e-6)
            # Eq. 8 by brute force: the budget's worth of largest priorities, ties to the lower position
            order = sorted(range(n + 1), key=lambda i: (-out["r"][i], i))[:5]
            np.testing.assert_array_equal(out["survivors"], sorted(order))
        ex = cam.export(with_kv=False)
        np.testing.assert_array_equal(ex["stored"], [norms[int(i)] for i in ex["ids"]])
    assert cam.evicted_total == 4


def test_camera_cache_config_rules():
    with pytest.raises(ValueError):                       # the budget must hold the first frame and K_max anchors
        orc.OracleLayer.camera(n_heads=1, head_dim=8, budget=3, k_max=3)
    orc.OracleLayer.camera(n_heads=1, head_dim=8, budget=4, k_max=3).close()
    with pytest.raises(ValueError):                       # a camera cache has no patch grid
        orc.OracleLayer(n_heads=1, head_dim=8, n_special=1, grid_h=2, grid_w=2, budget=16, anchor_tokens=0, camera_cache=1)
    agg = _tiny_layer()
    x = np.zeros((agg.M, agg.C), np.float32)
    agg.attend(0, x, x, x, compute=False)
    with pytest.raises(RuntimeError):                     # and the aggregator's cache is not a camera cache
        agg.compress_camera(np.zeros((1, agg.C), np.float32))


def test_create_rejects_budget_below_protected_bound():
    with pytest.raises(ValueError):
        _tiny_layer(budget=14 + 2 * 3 - 1)          # M + K_max * A = 20
    _tiny_layer(budget=20).close()


def test_attend_on_stream_equals_dense_attention_over_cache():
    cfg = gen.config_tiny().replace(budget=100)
    layer = orc.OracleLayer.from_stream(cfg)
    for t in range(3):
        fi = gen.frame_inputs(cfg, t)
        prev = layer.export()
        out = layer.attend(t, fi.q, fi.k, fi.v)
        Kall = np.concatenate([prev["k"], fi.k]); Vall = np.concatenate([prev["v"], fi.v])
        np.testing.assert_array_equal(out, orc.attention(fi.q, Kall, Vall, cfg.n_heads, cfg.head_dim))
        layer.compress(fi.resid, fi.conf, fi.rho)


def test_input_generator_is_reproducible_and_rounded():
    cfg = gen.config_tiny().replace(dtype=gen.DTYPE_BF16)
    a, b = gen.frame_inputs(cfg, 3), gen.frame_inputs(cfg, 3)
    assert np.array_equal(a.q, b.q) and np.array_equal(a.resid, b.resid) and a.rho == b.rho
    assert not np.array_equal(a.q, gen.frame_inputs(cfg, 4).q)
    bits = gen.bf16_round_bits(a.k)
    assert np.array_equal(gen.bf16_bits_to_f32(bits), a.k)          # already representable
    x = np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, np.nan], np.float32)   # ties to even
    np.testing.assert_array_equal(gen.bf16_round_bits(x)[:2], [0x3F80, 0x3F82])
    t = torch.from_numpy(a.q).to(torch.bfloat16).float().numpy()
    assert np.array_equal(t, a.q)
