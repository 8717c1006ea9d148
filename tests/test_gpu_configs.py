"""The other workload shapes, through the C ABI against the CPU oracle: the 518x392 token layout (1041 tokens),
a 24-layer handle, the budget / anchor sweep of the ultra-long stream in both score modes, and a 10,000-frame
soak that checks the invariants the method promises (constant cache size and memory, anchors never evicted,
flat per-frame time).  Streams are shortened where the oracle has to follow; the soak runs the library alone."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2603_05959_b200 import binding as B
from paper_2603_05959_b200 import inputs as gen
from paper_2603_05959_b200.stream import DeviceFrame, out_to_f32, storage_to_f32

pytestmark = pytest.mark.gpu

R_ATOL = 2e-5
R_RTOL_STORED = 2e-5       # fp32 fixed-order norms and smoothing against fp64
ATT_MAX, ATT_MEAN = 2e-2, 2e-3


def follow(cfg, n_frames, layers=(0,), attn_frames=(), attn_rows=None, export_at=(), threads=16):
    """Teacher-forced run of `n_frames` frames: the oracle follows the listed layers of one handle."""
    orc.set_threads(threads)
    cache = B.OvggtCache.from_stream(cfg)
    oracles = {l: orc.OracleLayer.from_stream(cfg) for l in layers}
    M = cfg.tokens_per_frame
    for t in range(n_frames):
        for l in range(cfg.n_layers):
            fi = gen.frame_inputs(cfg, t, layer=l)
            df = DeviceFrame(cfg, fi, "cuda")
            if l not in oracles:
                cache.layer_step(l, t, df.q, df.k, df.v, df.resid, df.conf, df.rho)
                continue
            o = oracles[l]
            check = t in attn_frames
            ref_out = o.attend(t, fi.q, fi.k, fi.v, rows=attn_rows, compute=check)
            ref = o.compress(fi.resid, fi.conf, fi.rho)
            out = cache.layer_attend(l, t, df.q, df.k, df.v)
            cache.layer_compress(l, t, df.resid, df.conf, df.rho, score_override=torch.from_numpy(ref["r"]).cuda())
            if check:
                got = out_to_f32(out)
                got = got if attn_rows is None else got[attn_rows]
                err = np.abs(got - ref_out)
                assert err.max() <= ATT_MAX and err.mean() <= ATT_MEAN, (t, l, err.max(), err.mean())
            sel = cache.last_selection(l)
            np.testing.assert_array_equal(sel["survivors"], ref["survivors"], err_msg=f"frame {t} layer {l}")
            fin = np.isfinite(ref["r"])
            # hybrid priorities lie in [0, 1]: absolute; stored residual norms are unnormalised: relative
            rtol, atol = (0, R_ATOL) if cfg.score_mode == gen.SCORE_HYBRID else (R_RTOL_STORED, 0)
            np.testing.assert_allclose(sel["r"][fin], ref["r"][fin], rtol=rtol, atol=atol, err_msg=f"frame {t} layer {l}")
            if t in export_at:
                ex, rx = cache.export(l), o.export()
                np.testing.assert_array_equal(ex["ids"], rx["ids"])
                np.testing.assert_array_equal(ex["flags"], rx["flags"])
                assert np.array_equal(storage_to_f32(ex["k"], cfg.dtype), rx["k"])
                assert np.array_equal(storage_to_f32(ex["v"], cfg.dtype), rx["v"])
        for l in range(cfg.n_layers):
            st = cache.stats(l)
            assert st["device_status"] == 0 and st["n_cached"] == min((t + 1) * M, cfg.budget)
            # Eq. 9
            assert st["n_protected_init"] + st["n_protected_hist"] <= M + cfg.k_max * cfg.anchor_tokens
    for l, o in oracles.items():
        st = cache.stats(l)
        assert st["anchor_frames"] == o.anchors() and st["evicted_total"] == o.evicted_total
    cache.destroy()
    return oracles


def test_aggregator_token_layout_1041_tokens():
    """518x392 frames: 37x28 patches + 5 = 1041 tokens (Sec. 3.1), budget 12288: fill, first evictions, an anchor."""
    cfg = gen.config_aggregator().replace(n_layers=1, min_anchor_interval=6, tau=0.7)
    assert cfg.tokens_per_frame == 1041
    rows = np.sort(np.random.default_rng(3).choice(1041, 12, replace=False)).astype(np.int32)
    o = follow(cfg, 16, attn_frames={0, 12, 15}, attn_rows=rows, export_at={13, 15})
    assert o[0].evicted_total > 0 and len(o[0].anchors()) >= 1


def test_stack_of_24_layers_each_with_its_own_cache():
    cfg = gen.config_stack24().replace(min_anchor_interval=3, tau=0.8)
    rows = np.array([0, 5, 700, 1373], dtype=np.int32)
    o = follow(cfg, 8, layers=(0, 11, 23), attn_frames={7}, attn_rows=rows, export_at={7})
    assert all(x.evicted_total > 0 for x in o.values())


def _follow_harness(model, cfg, n_frames, conf_rho, run_frame, rows):
    """Teacher-forced check of the library calls a workload harness makes: the oracle of every layer is fed the
    tensors the harness hands to the library (tap), its priorities are ranked on both sides, and the attention output
    (after) and the survivors are compared call by call."""
    orc.set_threads(16)
    oracles = [orc.OracleLayer.from_stream(cfg) for _ in range(cfg.n_layers)]
    pending, checked = {}, {"attn": 0, "sel": 0}

    def tap(t, l, q, k, v, resid):
        conf, rho = conf_rho(t)
        f32 = lambda x: x.float().cpu().numpy()
        ref_out = oracles[l].attend(t, f32(q), f32(k), f32(v), rows=rows)
        ref = oracles[l].compress(f32(resid), conf, rho)
        pending[(t, l)] = (ref_out, ref)
        return torch.from_numpy(ref["r"]).cuda()

    def after(t, l, out):
        pending[("out", t, l)] = out_to_f32(out)[rows]

    model.tap, model.after = tap, after
    for t in range(n_frames):
        run_frame(t)
        for l in range(cfg.n_layers):
            ref_out, ref = pending.pop((t, l))
            got = pending.pop(("out", t, l))
            err = np.abs(got - ref_out)
            assert err.max() <= ATT_MAX and err.mean() <= ATT_MEAN, (t, l, err.max(), err.mean())
            sel = model.cache.last_selection(l)
            np.testing.assert_array_equal(sel["survivors"], ref["survivors"], err_msg=f"frame {t} layer {l}")
            fin = np.isfinite(ref["r"])
            np.testing.assert_allclose(sel["r"][fin], ref["r"][fin], rtol=0, atol=R_ATOL, err_msg=f"frame {t} layer {l}")
            checked["attn"] += 1
            checked["sel"] += 1
            assert model.cache.stats(l)["device_status"] == 0
    for l, o in enumerate(oracles):
        ex, rx = model.cache.export(l), o.export()
        np.testing.assert_array_equal(ex["ids"], rx["ids"])
        np.testing.assert_array_equal(ex["flags"], rx["flags"])
        assert np.array_equal(storage_to_f32(ex["k"], cfg.dtype), rx["k"])
    return oracles, checked


def test_projection_stack_harness_library_calls_match_the_oracle():
    """The harness of the 24-layer workload (random-init QKV / output projections in torch around the library), cut
    to 3 layers and a budget that the frames overflow: every library call against the oracle."""
    from paper_2603_05959_b200 import harness as H
    cfg = gen.config_stack24().replace(n_layers=3, budget=3000, min_anchor_interval=2, tau=0.8)
    model = H.ProjectionStack(cfg, torch.device("cuda", torch.cuda.current_device()))
    stream = torch.cuda.current_stream()
    rows = np.array([0, 4, 5, 700, 1373], dtype=np.int32)

    def conf_rho(t):
        fi = gen.frame_inputs(cfg, t, fields=("anchor inputs only",))
        return fi.conf, fi.rho

    def run_frame(t):
        conf, rho, resid = H.frame_side_inputs(cfg, t, model.device, cfg.n_layers)
        model.frame(t, H.patch_embeddings(cfg, t, model.device), resid, conf, rho, stream)

    oracles, checked = _follow_harness(model, cfg, 5, conf_rho, run_frame, rows)
    assert checked["sel"] == 15 and all(o.evicted_total > 0 for o in oracles)
    model.destroy()


@pytest.mark.parametrize("batched", [True, False], ids=["compress-all-layers-at-frame-end", "compress-per-layer"])
def test_aggregator_harness_library_calls_match_the_oracle(batched):
    """The alternating-aggregator harness (frame attention and MLPs in torch; attend -> MLP -> compress around the
    library, the activation score fed by the block's real MLP output), cut to 2 depths: every library call against
    the oracle, on the 1041-token layout."""
    from paper_2603_05959_b200 import harness as H
    cfg = gen.config_aggregator().replace(n_layers=2, budget=2500, min_anchor_interval=2, tau=0.8)
    model = H.Aggregator(cfg, torch.device("cuda", torch.cuda.current_device()), batched_compress=batched)
    stream = torch.cuda.current_stream()
    rows = np.array([0, 3, 5, 512, 1040], dtype=np.int32)

    def conf_rho(t):
        fi = gen.frame_inputs(cfg, t, fields=("anchor inputs only",))
        return fi.conf, fi.rho

    def run_frame(t):
        conf, rho, _ = H.frame_side_inputs(cfg, t, model.device, 0)
        model.frame(t, H.patch_embeddings(cfg, t, model.device), conf, rho, stream)

    oracles, checked = _follow_harness(model, cfg, 5, conf_rho, run_frame, rows)
    assert checked["sel"] == 10 and all(o.evicted_total > 0 for o in oracles)
    model.destroy()


@pytest.mark.parametrize("budget,anchors,mode,frames", [
    (4096, 0, gen.SCORE_HYBRID, 12),
    (4096, 256, gen.SCORE_RESIDUAL_STORED, 12),
    (32768, 256, gen.SCORE_HYBRID, 27),
    (32768, 64, gen.SCORE_RESIDUAL_STORED, 27),
])
def test_ultra_long_sweep_points(budget, anchors, mode, frames):
    cfg = gen.config_ultra_long(budget, anchors, mode).replace(min_anchor_interval=5, tau=0.6)
    rows = np.array([3, 640, 1370], dtype=np.int32)
    o = follow(cfg, frames, attn_frames={frames - 1}, attn_rows=rows, export_at={frames - 1})
    assert o[0].evicted_total > 0


def test_soak_10000_frames_constant_cost_and_invariants():
    """10,000 frames through one layer (budget 4096, 64 anchor tokens, drifting residual gain): the cache size,
    the device memory and the per-frame time stay constant, first-frame rows and active anchors are never
    evicted, ids stay ascending, and the device status word stays clear."""
    cfg = gen.config_ultra_long(4096, 64)
    M, Bud = cfg.tokens_per_frame, cfg.budget
    cache = B.OvggtCache.from_stream(cfg)
    out = cache.new_out()
    stream = torch.cuda.current_stream()
    pool = {}

    def block_frames(block):          # 12 distinct frames per block of 1000, drawn at that block's gain level
        if block not in pool:
            pool.clear()
            pool[block] = [DeviceFrame(cfg, gen.frame_inputs(cfg, block * 1000 + i), "cuda") for i in range(12)]
        return pool[block]

    block_frames(0)
    torch.cuda.synchronize()
    mem0 = torch.cuda.memory_allocated()
    times = []
    for block in range(10):
        fr = block_frames(block)
        torch.cuda.synchronize()
        mem_block = torch.cuda.memory_allocated()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(1000):
            t = block * 1000 + i
            f = fr[i % len(fr)]
            cache.layer_step(0, t, f.q, f.k, f.v, f.resid, f.conf, f.rho, out=out, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() <= mem_block          # the steps allocate nothing
        times.append(e0.elapsed_time(e1) / 1000.0)
        st = cache.stats(0)
        assert st["device_status"] == 0 and st["n_cached"] == Bud and st["frames_seen"] == (block + 1) * 1000
        assert st["bytes_resident"] == 2 * (Bud + M) * cfg.dim * cfg.elem_bytes      # one K and one V buffer
        assert st["n_protected_init"] == M and st["n_protected_hist"] == cfg.anchor_tokens * st["n_active_anchors"]
        assert st["n_active_anchors"] <= cfg.k_max
        ex = cache.export(0, with_kv=False)
        ids, flags = ex["ids"], ex["flags"]
        assert len(ids) == Bud and np.all(np.diff(ids) > 0)
        assert np.array_equal(ids[:M], np.arange(M)) and np.all(flags[:M] == B.FLAG_INIT)   # the first frame, for good
        hist_frames = sorted(set((ids[flags == B.FLAG_HIST] // M).tolist()))
        assert hist_frames == st["anchor_frames"]
        assert int((flags == B.FLAG_HIST).sum()) == st["n_protected_hist"]
        if block > 0:                                               # consecutive anchors are >= 100 frames apart
            af = st["anchor_frames"]
            assert all(b - a >= cfg.min_anchor_interval for a, b in zip(af, af[1:]))
    assert bool(torch.isfinite(out.float()).all())
    steady = np.array(times[1:])                                    # block 0 contains the fill phase
    assert steady.max() / np.median(steady) < 1.15, times
    assert torch.cuda.memory_allocated() <= mem0 + 64 * 1024 * 1024
    cache.destroy()
