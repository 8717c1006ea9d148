"""Stream parity: the library (through the C ABI) against the CPU oracle on the same seeded frames.

Protocol: the oracle runs freely; the library is teacher-forced with the oracle's fp32 priorities, so the
survivor sets and the cache layout must be bit-exact, while the library's own priorities are compared
with a tolerance.  A second test lets the library run freely and requires any divergence to be a near-tie."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2603_05959_b200 import binding as B
from paper_2603_05959_b200 import inputs as gen
from paper_2603_05959_b200.stream import DeviceFrame, out_to_f32, storage_to_f32

from attn_cases import assert_attention_close_relative, sampled_rows_all_groups, tiled_hot_case

pytestmark = pytest.mark.gpu

R_ATOL = 2e-5          # priorities live in [0, 0.5]; fp32 scores after min-max against fp64
STORED_RTOL = 2e-5
ATT_MAX, ATT_MEAN, ATT_F32 = 2e-2, 2e-3, 1e-4


def run_teacher_forced(cfg, n_frames, attn_frames, attn_rows=None, export_every=1, threads=8,
                       compaction=B.COMPACT_FILL_HOLES, r_atol=R_ATOL, stored_rtol=STORED_RTOL):
    orc.set_threads(threads)
    layer = orc.OracleLayer.from_stream(cfg)
    cache = B.OvggtCache.from_stream(cfg.replace(n_layers=1), compaction=compaction)
    M, Bud = cfg.tokens_per_frame, cfg.budget
    for t in range(n_frames):
        fi = gen.frame_inputs(cfg, t)
        df = DeviceFrame(cfg, fi, "cuda")
        check_attn = t in attn_frames
        ref_out = layer.attend(t, fi.q, fi.k, fi.v, rows=attn_rows, compute=check_attn)
        ref = layer.compress(fi.resid, fi.conf, fi.rho)
        out = cache.layer_attend(0, t, df.q, df.k, df.v)
        ov = torch.from_numpy(ref["r"]).cuda()
        cache.layer_compress(0, t, df.resid, df.conf, df.rho, score_override=ov)
        if check_attn:
            got = out_to_f32(out)
            got = got if attn_rows is None else got[attn_rows]
            err = np.abs(got - ref_out)
            if cfg.dtype == gen.DTYPE_F32:
                assert err.max() <= ATT_F32, (t, err.max())
            else:
                assert err.max() <= ATT_MAX and err.mean() <= ATT_MEAN, (t, err.max(), err.mean())
        sel = cache.last_selection(0)
        np.testing.assert_array_equal(sel["survivors"], ref["survivors"], err_msg=f"frame {t}")
        fin = np.isfinite(ref["r"])
        assert np.array_equal(np.isinf(sel["r"]), ~fin), t
        np.testing.assert_allclose(sel["r"][fin], ref["r"][fin], rtol=0, atol=r_atol, err_msg=f"frame {t}")
        st = cache.stats(0)
        assert st["n_cached"] == layer.n_rows == min(st["last_n_candidates"], Bud)
        assert st["device_status"] == 0
        n_init, n_hist = layer.protected()
        assert (st["n_protected_init"], st["n_protected_hist"]) == (n_init, n_hist)
        assert st["anchor_frames"] == layer.anchors()
        assert st["evicted_total"] == layer.evicted_total
        if t % export_every == 0 or t == n_frames - 1:
            ex, rx = cache.export(0), layer.export()
            np.testing.assert_array_equal(ex["ids"], rx["ids"])
            np.testing.assert_array_equal(ex["flags"], rx["flags"])
            if cfg.score_mode == gen.SCORE_QK:
                # a sum of signed products: fp32 rounding scales with the largest score, not with one that cancels
                np.testing.assert_allclose(ex["stored"], rx["stored"], rtol=0,
                                           atol=stored_rtol * float(np.abs(rx["stored"]).max()))
            else:
                np.testing.assert_allclose(ex["stored"], rx["stored"], rtol=stored_rtol)
            assert np.array_equal(storage_to_f32(ex["k"], cfg.dtype), rx["k"])
            assert np.array_equal(storage_to_f32(ex["v"], cfg.dtype), rx["v"])
    bytes0 = cache.stats(0)["bytes_resident"]
    buffers = 1 if compaction == B.COMPACT_FILL_HOLES else 2       # (K and V) x buffers x (B + M) rows
    assert bytes0 == 2 * buffers * (Bud + M) * cfg.dim * cfg.elem_bytes
    cache.destroy()
    return layer


BOTH_LAYOUTS = pytest.mark.parametrize("compaction", [B.COMPACT_FILL_HOLES, B.COMPACT_STABLE_GATHER])


@BOTH_LAYOUTS
def test_config1_tiny_fp32_every_frame(compaction):
    cfg = gen.config_tiny()
    layer = run_teacher_forced(cfg, cfg.n_frames, attn_frames=set(range(cfg.n_frames)), compaction=compaction)
    assert layer.evicted_total > 0 and len(layer.anchors()) >= 1


def test_hole_filling_column_sums_follow_the_cache_across_refreshes():
    """In the hole-filling layout the key column sums behind the diversity score are continued from step to step
    (+ admitted keys - evicted keys) and summed afresh every 64th step.  150 frames of the tiny stream cross two
    refreshes; the library's own priorities are compared with the oracle's on every frame (run_teacher_forced), so
    drift between refreshes, or a wrong correction, shows up as a priority off by more than the tolerance."""
    cfg = gen.config_tiny().replace(n_frames=150, min_anchor_interval=20)
    layer = run_teacher_forced(cfg, cfg.n_frames, attn_frames={0, 70, 149}, export_every=25)
    assert layer.evicted_total > 100 * cfg.tokens_per_frame


def test_config1_frequent_anchors_exercise_fifo_demotion():
    cfg = gen.config_tiny().replace(tau=0.95, min_anchor_interval=2, k_max=2, n_frames=14)
    layer = run_teacher_forced(cfg, cfg.n_frames, attn_frames={0, 5, 13})
    assert len(layer.anchors()) == 2


def test_stored_residual_mode_and_no_anchors():
    cfg = gen.config_tiny().replace(score_mode=gen.SCORE_RESIDUAL_STORED, anchor_tokens=0, budget=200)
    run_teacher_forced(cfg, 10, attn_frames={9})
    cfg = gen.config_tiny().replace(protect_first_frame=0, budget=100, beta=0.8, alpha=0.0)
    run_teacher_forced(cfg, 8, attn_frames={7})


def test_random_eviction_mode_runs_free_and_matches_the_oracle_bit_for_bit():
    """The random-eviction baseline (Supp. A).  Its priorities are counter-based values that both sides compute
    from (seed, frame, token id) exactly, so no teacher forcing is needed: the library runs freely and must keep the
    oracle's survivors, priorities and layout bit for bit, in both layouts."""
    cfg = gen.StreamConfig(name="rnd", n_heads=2, grid_h=7, grid_w=9, budget=250, anchor_tokens=5, k_max=2,
                           min_anchor_interval=3, tau=0.9, n_frames=25, dtype=gen.DTYPE_F32, score_mode=gen.SCORE_RANDOM)
    for compaction in (B.COMPACT_FILL_HOLES, B.COMPACT_STABLE_GATHER):
        layer = orc.OracleLayer.from_stream(cfg)
        c = B.OvggtCache.from_stream(cfg, compaction=compaction)
        for t in range(cfg.n_frames):
            fi = gen.frame_inputs(cfg, t)
            df = DeviceFrame(cfg, fi, "cuda")
            layer.attend(t, fi.q, fi.k, fi.v, compute=False)
            ref = layer.compress(fi.resid, fi.conf, fi.rho)
            c.layer_step(0, t, df.q, df.k, df.v, df.resid, df.conf, df.rho)
            sel = c.last_selection(0)
            np.testing.assert_array_equal(sel["survivors"], ref["survivors"], err_msg=f"frame {t}")
            np.testing.assert_array_equal(sel["r"], ref["r"], err_msg=f"frame {t}")
        ex, rx = c.export(0), layer.export()
        np.testing.assert_array_equal(ex["ids"], rx["ids"])
        np.testing.assert_array_equal(ex["flags"], rx["flags"])
        assert np.array_equal(ex["k"], rx["k"]) and layer.evicted_total > 0
        c.destroy()


@BOTH_LAYOUTS
def test_query_key_mode_matches_the_oracle(compaction):
    """The query-key criterion of the scoring probe (Supp. D) in place of Eq. 5: the library's own priorities of the
    new rows (mean scaled logit through the column sums of Q, smoothed, min-max normalised) against the oracle's
    triple loop on every frame, fp32 and bf16, anchors on; survivors and layout bit-exact under teacher forcing."""
    cfg = gen.config_tiny().replace(score_mode=gen.SCORE_QK, n_frames=14, min_anchor_interval=4)
    layer = run_teacher_forced(cfg, cfg.n_frames, attn_frames={13}, compaction=compaction)
    assert layer.evicted_total > 0
    mid = gen.StreamConfig(name="qk", n_heads=2, grid_h=13, grid_w=11, budget=600, anchor_tokens=7,
                           min_anchor_interval=3, tau=0.5, n_frames=10, score_mode=gen.SCORE_QK)
    run_teacher_forced(mid, mid.n_frames, attn_frames={9}, export_every=3, compaction=compaction)


def test_query_key_mode_through_the_overlapped_step_and_the_batched_compress():
    """The same criterion on the other two routes into the selection: ovggt_layer_step (scores on the side stream,
    no residual given at all) and attend-per-layer followed by one ovggt_layers_compress for two layers, where each
    layer's scores wait in the layer's own buffer."""
    cfg = gen.config_tiny().replace(score_mode=gen.SCORE_QK, n_frames=12, n_layers=2)
    ora = [orc.OracleLayer.from_stream(cfg) for _ in range(2)]
    step, split = B.OvggtCache.from_stream(cfg), B.OvggtCache.from_stream(cfg)
    for t in range(cfg.n_frames):
        fis = [gen.frame_inputs(cfg, t, layer=l) for l in range(2)]
        dfs = [DeviceFrame(cfg, fi, "cuda") for fi in fis]
        refs = []
        for l in range(2):
            ora[l].attend(t, fis[l].q, fis[l].k, fis[l].v, compute=False)
            refs.append(ora[l].compress(None, fis[l].conf, fis[l].rho))
        ovs = [torch.from_numpy(r["r"]).cuda() for r in refs]
        for l in range(2):
            step.layer_step(l, t, dfs[l].q, dfs[l].k, dfs[l].v, None, dfs[l].conf, dfs[l].rho, score_override=ovs[l])
            split.layer_attend(l, t, dfs[l].q, dfs[l].k, dfs[l].v)
        split.layers_compress(t, [None, None], conf=dfs[0].conf, rho=dfs[0].rho, score_overrides=ovs)
        for cache in (step, split):
            for l in range(2):
                sel = cache.last_selection(l)
                np.testing.assert_array_equal(sel["survivors"], refs[l]["survivors"], err_msg=f"frame {t} layer {l}")
                fin = np.isfinite(refs[l]["r"])
                np.testing.assert_allclose(sel["r"][fin], refs[l]["r"][fin], rtol=0, atol=R_ATOL)
    assert ora[0].evicted_total > 0
    for cache in (step, split):
        assert cache.stats(0)["device_status"] == 0
        cache.destroy()


def test_largest_budget_the_selection_cluster_holds():
    """Maximum size.  The fused selection kernel keeps all B + M candidates of a layer in the shared memory of one
    8-CTA cluster; ovggt_cache_create refuses a budget beyond that with OVGGT_ERR_UNSUPPORTED.  The largest budget it
    accepts for 2000-token frames (found by asking) is filled and then evicts for five frames, teacher-forced:
    survivors and layout bit-exact, the library's own priorities within tolerance, at about 75,000 candidates."""
    base = gen.StreamConfig(name="max", n_heads=1, n_special=20, grid_h=45, grid_w=44, anchor_tokens=16,
                            min_anchor_interval=5, tau=0.6, budget=0)

    def accepted(budget):
        try:
            B.OvggtCache.from_stream(base.replace(budget=budget)).destroy()
            return True
        except B.OvggtError as e:
            assert e.code == B.ERR_UNSUPPORTED, e
            return False

    lo, hi = 40_000, 200_000                    # accepted, refused
    assert accepted(lo) and not accepted(hi)
    while hi - lo > 500:
        mid = (lo + hi) // 2
        lo, hi = (mid, hi) if accepted(mid) else (lo, mid)
    assert 60_000 <= lo <= 100_000, lo
    cfg = base.replace(budget=lo, n_frames=lo // base.tokens_per_frame + 6)
    layer = run_teacher_forced(cfg, cfg.n_frames, attn_frames=set(), export_every=10_000)
    assert layer.evicted_total >= 4 * cfg.tokens_per_frame and layer.n_rows == lo


@BOTH_LAYOUTS
def test_attention_weight_mode_matches_the_oracle(compaction):
    """The attention-weight criterion of the scoring probe (Supp. D): the attention the frame's tokens receive in
    the frame's own attention, from the attention kernels' log2 denominators and a second pass over the frame's
    M x M block, against the oracle's materialised softmax on every frame; fp32 (SIMT attention) and bf16 (tcgen05
    attention, split and merged).  In bf16 a third of the attention kernel's exponentials are cubics of relative
    error 1e-4, which enters every denominator: scores and priorities are compared at 5e-4 of their range there."""
    cfg = gen.config_tiny().replace(score_mode=gen.SCORE_ATTN, n_frames=12, min_anchor_interval=4)
    layer = run_teacher_forced(cfg, cfg.n_frames, attn_frames={11}, compaction=compaction)
    assert layer.evicted_total > 0
    mid = gen.StreamConfig(name="aw", n_heads=2, grid_h=13, grid_w=11, budget=600, anchor_tokens=7,
                           min_anchor_interval=3, tau=0.5, n_frames=8, score_mode=gen.SCORE_ATTN)
    run_teacher_forced(mid, mid.n_frames, attn_frames={7}, export_every=3, compaction=compaction, r_atol=2.5e-4,
                       stored_rtol=5e-4)


def test_attention_weight_mode_through_layer_step_without_a_residual():
    cfg = gen.config_tiny().replace(score_mode=gen.SCORE_ATTN, n_frames=10)
    ora = orc.OracleLayer.from_stream(cfg)
    cache = B.OvggtCache.from_stream(cfg)
    for t in range(cfg.n_frames):
        fi = gen.frame_inputs(cfg, t)
        df = DeviceFrame(cfg, fi, "cuda")
        ora.attend(t, fi.q, fi.k, fi.v, compute=False)
        ref = ora.compress(None, fi.conf, fi.rho)
        cache.layer_step(0, t, df.q, df.k, df.v, None, df.conf, df.rho, score_override=torch.from_numpy(ref["r"]).cuda())
        sel = cache.last_selection(0)
        np.testing.assert_array_equal(sel["survivors"], ref["survivors"], err_msg=f"frame {t}")
        fin = np.isfinite(ref["r"])
        np.testing.assert_allclose(sel["r"][fin], ref["r"][fin], rtol=0, atol=R_ATOL)
    assert ora.evicted_total > 0 and cache.stats(0)["device_status"] == 0
    cache.destroy()


@BOTH_LAYOUTS
def test_bf16_ragged_midsize_stream(compaction):
    """Several KV tiles with a ragged tail, two ragged query tiles, bf16, anchors on."""
    cfg = gen.StreamConfig(name="mid", n_heads=2, grid_h=13, grid_w=11, budget=600, anchor_tokens=7,
                           min_anchor_interval=3, tau=0.5, n_frames=12)
    run_teacher_forced(cfg, cfg.n_frames, attn_frames=set(range(12)), compaction=compaction)


def test_budget_not_a_multiple_of_the_frame_and_demotions_in_the_hole_filling_layout():
    """A budget that the frames do not fill evenly (the first eviction step has new rows on both sides of slot B)
    and frequent anchor turnover, stored-score mode included: layouts must still export in token order."""
    cfg = gen.StreamConfig(name="odd", n_heads=2, grid_h=6, grid_w=7, budget=131, anchor_tokens=5, k_max=2,
                           min_anchor_interval=2, tau=0.9, n_frames=20, dtype=gen.DTYPE_F32)
    run_teacher_forced(cfg, cfg.n_frames, attn_frames={0, 3, 19})
    run_teacher_forced(cfg.replace(score_mode=gen.SCORE_RESIDUAL_STORED), cfg.n_frames, attn_frames={19})


def test_free_running_divergence_is_only_a_near_tie():
    cfg = gen.config_tiny()
    layer = orc.OracleLayer.from_stream(cfg)
    cache = B.OvggtCache.from_stream(cfg)
    for t in range(cfg.n_frames):
        fi = gen.frame_inputs(cfg, t)
        df = DeviceFrame(cfg, fi, "cuda")
        layer.attend(t, fi.q, fi.k, fi.v, compute=False)
        ref = layer.compress(fi.resid, fi.conf, fi.rho)
        cache.layer_step(0, t, df.q, df.k, df.v, df.resid, df.conf, df.rho)
        sel = cache.last_selection(0)
        if not np.array_equal(sel["survivors"], ref["survivors"]):
            a, b = set(sel["survivors"].tolist()), set(ref["survivors"].tolist())
            diff = sorted(a ^ b)
            kth = np.sort(ref["r"][np.isfinite(ref["r"])])[::-1][cfg.budget - int(np.isinf(ref["r"]).sum()) - 1]
            assert all(abs(ref["r"][i] - kth) <= R_ATOL for i in diff), (t, diff)
            break
    cache.destroy()


def same_output(oa, ob, compaction):
    """Two handles that hold the same cache.  With the stable gather both hold it in token order and every sum runs
    in the same order: bit-identical outputs.  With hole filling an imported cache lies in token order while the
    handle it came from holds the same rows in slot order, so the attention adds the same terms in another order:
    equal to fp32 rounding of an fp32 accumulation."""
    if compaction == B.COMPACT_STABLE_GATHER:
        return torch.equal(oa, ob)
    return bool(torch.allclose(oa.float(), ob.float(), rtol=0, atol=2e-6 if oa.dtype == torch.float32 else 2e-2))


@BOTH_LAYOUTS
def test_export_import_roundtrip_and_resume(compaction):
    cfg = gen.config_tiny().replace(n_frames=10)
    a = B.OvggtCache.from_stream(cfg, compaction=compaction)
    frames = [DeviceFrame(cfg, gen.frame_inputs(cfg, t), "cuda") for t in range(cfg.n_frames)]
    for t in range(6):
        f = frames[t]
        a.layer_step(0, t, f.q, f.k, f.v, f.resid, f.conf, f.rho)
    ex = a.export(0)
    st = a.stats(0)
    b = B.OvggtCache.from_stream(cfg, compaction=compaction)
    last_reg = st["anchor_frames"][-1] if st["anchor_frames"] else 0
    b.import_(0, ex["ids"], ex["flags"], ex["stored"], ex["k"], ex["v"], next_frame_id=6, last_registration_frame=last_reg)
    ex2 = b.export(0)
    for key in ex:
        assert np.array_equal(ex[key], ex2[key])
    for t in range(6, 10):
        f = frames[t]
        oa = a.layer_step(0, t, f.q, f.k, f.v, f.resid, f.conf, f.rho)
        ob = b.layer_step(0, t, f.q, f.k, f.v, f.resid, f.conf, f.rho)
        assert same_output(oa, ob, compaction)
    ea, eb = a.export(0), b.export(0)
    for key in ea:
        assert np.array_equal(ea[key], eb[key])
    a.destroy(); b.destroy()


@BOTH_LAYOUTS
def test_two_layer_export_import_resume_and_anchor_state_rules(compaction):
    """The anchor FIFO belongs to the handle.  Two layers are exported in the middle of a stream with active
    anchors, imported into a fresh handle (the first import brings the handle-wide state, the second must agree
    with it) and both handles continue bit-identically.  Imports that disagree, and an empty import, leave the
    handle-wide state untouched."""
    cfg = gen.config_tiny().replace(n_layers=2, n_frames=12, tau=0.9, min_anchor_interval=2, k_max=2)
    a = B.OvggtCache.from_stream(cfg, compaction=compaction)
    frames = [[DeviceFrame(cfg, gen.frame_inputs(cfg, t, layer=l), "cuda") for l in range(2)] for t in range(cfg.n_frames)]

    def step(c, t):
        return [c.layer_step(l, t, f.q, f.k, f.v, f.resid, f.conf, f.rho) for l, f in enumerate(frames[t])]

    for t in range(7):
        step(a, t)
    ex = [a.export(l) for l in range(2)]
    sa = a.stats(0)
    assert sa["n_active_anchors"] == 2                      # the FIFO is in use when the state is moved
    last_reg = sa["anchor_frames"][-1]
    b = B.OvggtCache.from_stream(cfg, compaction=compaction)
    b.import_(0, ex[0]["ids"], ex[0]["flags"], ex[0]["stored"], ex[0]["k"], ex[0]["v"], 7, last_reg)
    # an empty import of the other layer must not wipe what layer 0 brought
    b.import_(1, ex[1]["ids"][:0], ex[1]["flags"][:0], ex[1]["stored"][:0], ex[1]["k"][:0], ex[1]["v"][:0], 7, last_reg)
    assert b.stats(0)["anchor_frames"] == sa["anchor_frames"]
    # a layer whose HIST rows name other frames than the handle's FIFO is refused
    bad_flags = ex[1]["flags"].copy()
    bad_flags[bad_flags == B.FLAG_HIST] = B.FLAG_EVICTABLE
    with pytest.raises(B.OvggtError) as e:
        b.import_(1, ex[1]["ids"], bad_flags, ex[1]["stored"], ex[1]["k"], ex[1]["v"], 7, last_reg)
    assert e.value.code == -1
    with pytest.raises(B.OvggtError):
        b.import_(1, ex[1]["ids"], ex[1]["flags"], ex[1]["stored"], ex[1]["k"], ex[1]["v"], 7, last_reg - 1)
    b.import_(1, ex[1]["ids"], ex[1]["flags"], ex[1]["stored"], ex[1]["k"], ex[1]["v"], 7, last_reg)
    for l in range(2):
        sb = b.stats(l)
        assert sb["anchor_frames"] == sa["anchor_frames"]
        assert (sb["n_protected_init"], sb["n_protected_hist"]) == (a.stats(l)["n_protected_init"], a.stats(l)["n_protected_hist"])
    for t in range(7, cfg.n_frames):
        for oa, ob in zip(step(a, t), step(b, t)):
            assert same_output(oa, ob, compaction)
    for l in range(2):
        ea, eb = a.export(l), b.export(l)
        for key in ea:
            assert np.array_equal(ea[key], eb[key]), (l, key)
        assert a.stats(l)["anchor_frames"] == b.stats(l)["anchor_frames"]
    # reset empties the handle, after which another stream can be imported
    b.reset()
    assert b.stats(0)["n_cached"] == 0 and b.stats(0)["anchor_frames"] == []
    b.import_(0, ex[0]["ids"], ex[0]["flags"], ex[0]["stored"], ex[0]["k"], ex[0]["v"], 7, last_reg)
    assert b.stats(0)["anchor_frames"] == sa["anchor_frames"]
    a.destroy(); b.destroy()


def test_layers_must_compress_frames_in_order_across_the_handle():
    """Layer 0 runs one frame ahead; layer 1 then comes with the older frame.  Its compress is refused (the anchor
    decision of that frame cannot be taken twice) and the anchor state is what layer 0 left."""
    cfg = gen.config_tiny().replace(n_layers=2, tau=0.95, min_anchor_interval=1, k_max=2)
    c = B.OvggtCache.from_stream(cfg)
    f = [[DeviceFrame(cfg, gen.frame_inputs(cfg, t, layer=l), "cuda") for l in range(2)] for t in range(4)]
    for t in range(2):
        for l in range(2):
            x = f[t][l]
            c.layer_step(l, t, x.q, x.k, x.v, x.resid, x.conf, x.rho)
    x = f[2][0]
    c.layer_attend(0, 2, x.q, x.k, x.v)
    y = f[2][1]
    c.layer_attend(1, 2, y.q, y.k, y.v)
    c.layer_compress(0, 2, x.resid, x.conf, x.rho)
    x3 = f[3][0]
    c.layer_step(0, 3, x3.q, x3.k, x3.v, x3.resid, x3.conf, x3.rho)      # layer 0 is now ahead of layer 1
    before = c.stats(0)["anchor_frames"]
    with pytest.raises(B.OvggtError) as e:
        c.layer_compress(1, 2, y.resid, y.conf, y.rho)
    assert e.value.code == -4
    assert c.stats(0)["anchor_frames"] == before
    c.destroy()


def test_bounded_device_wait_runs_out_cleanly_and_the_handle_recovers():
    """Failure detection without a fault: the wait routine of the attention kernel is run on a barrier that nothing
    completes, with a 2 ms limit.  The kernel returns, the status word and ovggt_cache_stats report the time-out,
    the context stays usable, and after clearing the status the same handle passes a teacher-forced step."""
    cfg = gen.config_tiny()
    c = B.OvggtCache.from_stream(cfg)
    layer = orc.OracleLayer.from_stream(cfg)

    def forced_step(t):
        fi = gen.frame_inputs(cfg, t)
        df = DeviceFrame(cfg, fi, "cuda")
        ref_out = layer.attend(t, fi.q, fi.k, fi.v)
        ref = layer.compress(fi.resid, fi.conf, fi.rho)
        out = c.layer_step(0, t, df.q, df.k, df.v, df.resid, df.conf, df.rho, score_override=torch.from_numpy(ref["r"]).cuda())
        assert np.abs(out_to_f32(out) - ref_out).max() <= ATT_F32
        np.testing.assert_array_equal(c.last_selection(0)["survivors"], ref["survivors"])

    forced_step(0)
    assert c.stats(0)["device_status"] == 0
    waited = c.selftest_bounded_wait(2000)
    assert 2_000_000 <= waited < 200_000_000                 # gave up after the limit, long before the default second
    with pytest.raises(B.OvggtError) as e:
        c.stats(0)
    assert e.value.code == -9                                  # OVGGT_ERR_TIMEOUT, surfaced by the next stats call
    torch.cuda.synchronize()                                   # the context is intact
    c.clear_status()
    for t in range(1, 6):
        forced_step(t)
    assert c.stats(0)["device_status"] == 0
    c.destroy()


def test_call_order_errors():
    cfg = gen.config_tiny()
    c = B.OvggtCache.from_stream(cfg)
    f = DeviceFrame(cfg, gen.frame_inputs(cfg, 0), "cuda")
    with pytest.raises(B.OvggtError) as e:
        c.layer_compress(0, 0, f.resid)                    # nothing appended yet
    assert e.value.code == -4
    c.layer_attend(0, 0, f.q, f.k, f.v)
    with pytest.raises(B.OvggtError):
        c.layer_attend(0, 1, f.q, f.k, f.v)                # previous frame not compressed
    with pytest.raises(B.OvggtError):
        c.layer_compress(0, 3, f.resid)                    # wrong frame id
    c.layer_compress(0, 0, f.resid, f.conf, f.rho)
    with pytest.raises(B.OvggtError):
        c.layer_attend(0, 0, f.q, f.k, f.v)                # frame ids must increase
    with pytest.raises(B.OvggtError) as e:
        c.layer_attend(3, 1, f.q, f.k, f.v)
    assert e.value.code == -2
    with pytest.raises(B.OvggtError) as e:
        c.layer_attend(0, 1, f.q.view(-1)[1:].view(-1), f.k, f.v)   # misaligned pointer
    assert e.value.code == -5
    assert c.stats(0)["device_status"] == 0
    c.destroy()


@pytest.mark.parametrize("pin", [True, False])
def test_host_buffer_entry_point_matches_device_entry_point(pin):
    """Pinned buffers: staged copies on the handle's copy stream, output written by the kernel into host memory.
    Pageable buffers: the output comes back through the staging buffer.  Several calls are in flight before the
    first synchronisation, so both staging sets are in use."""
    cfg = gen.StreamConfig(name="mid", n_heads=2, grid_h=9, grid_w=10, budget=300, anchor_tokens=4,
                           min_anchor_interval=2, tau=0.5, n_frames=7)
    a, b = B.OvggtCache.from_stream(cfg), B.OvggtCache.from_stream(cfg)
    host = [DeviceFrame(cfg, gen.frame_inputs(cfg, t), None, pin=pin) for t in range(cfg.n_frames)]
    outs_b = []
    for t in range(cfg.n_frames):                        # no synchronisation between the calls
        h = host[t]
        ob = torch.empty((cfg.tokens_per_frame, cfg.dim), dtype=torch.bfloat16)
        ob = ob.pin_memory() if pin else ob
        b.layer_step_host(0, t, h.q, h.k, h.v, h.resid, h.conf, h.rho, ob)
        outs_b.append(ob)
    torch.cuda.synchronize()
    for t in range(cfg.n_frames):
        fi = gen.frame_inputs(cfg, t)
        d = DeviceFrame(cfg, fi, "cuda")
        oa = a.layer_step(0, t, d.q, d.k, d.v, d.resid, d.conf, d.rho)
        torch.cuda.synchronize()
        assert torch.equal(oa.cpu(), outs_b[t]), t
    ea, eb = a.export(0), b.export(0)
    for key in ea:
        assert np.array_equal(ea[key], eb[key])
    a.destroy(); b.destroy()


def test_multi_layer_handle_shares_the_anchor_decision():
    cfg = gen.config_tiny().replace(n_layers=3, tau=0.9, n_frames=8)
    c = B.OvggtCache.from_stream(cfg)
    oracles = [orc.OracleLayer.from_stream(cfg) for _ in range(3)]
    for t in range(cfg.n_frames):
        for l in range(3):
            fi = gen.frame_inputs(cfg, t, layer=l)
            d = DeviceFrame(cfg, fi, "cuda")
            oracles[l].attend(t, fi.q, fi.k, fi.v, compute=False)
            ref = oracles[l].compress(fi.resid, fi.conf, fi.rho)
            c.layer_step(0 + l, t, d.q, d.k, d.v, d.resid, d.conf, d.rho, score_override=torch.from_numpy(ref["r"]).cuda())
            np.testing.assert_array_equal(c.last_selection(l)["survivors"], ref["survivors"])
        for l in range(3):
            assert c.stats(l)["anchor_frames"] == oracles[l].anchors()
    c.destroy()


@BOTH_LAYOUTS
def test_config2_full_size_stream_teacher_forced(compaction):
    """The benchmark configuration itself (1374 tokens/frame, budget 16384, bf16): 40 frames cover the
    fill phase, the first evictions and steady state; attention is checked on sampled rows."""
    cfg = gen.config_vggt_layer()
    rows = np.sort(np.random.default_rng(11).choice(cfg.tokens_per_frame, 16, replace=False)).astype(np.int32)
    threads = max(1, min(32, torch.get_num_threads()))
    run_teacher_forced(cfg, 40, attn_frames={0, 11, 12, 39}, attn_rows=rows, export_every=13, threads=threads,
                       compaction=compaction)


@pytest.mark.parametrize("dtype,compaction", [(gen.DTYPE_F32, B.COMPACT_FILL_HOLES), (gen.DTYPE_BF16, B.COMPACT_FILL_HOLES),
                                              (gen.DTYPE_F32, B.COMPACT_STABLE_GATHER)])
def test_all_layers_compressed_in_one_call_with_per_layer_budgets(dtype, compaction):
    """ovggt_layers_compress: three layers with budgets of their own (Sec. 3.2), attended one by one and compressed
    together - the way a model works whose anchor inputs exist only after its heads.  Teacher-forced per layer, so
    survivors, priorities, counters and exported layouts must match three independent oracles frame by frame."""
    budgets = [256, 150, 333]
    cfg = gen.config_tiny().replace(n_layers=3, tau=0.9, min_anchor_interval=2, k_max=2, n_frames=14, dtype=dtype)
    c = B.OvggtCache.from_stream(cfg, budget=budgets, compaction=compaction)
    oracles = [orc.OracleLayer.from_stream(cfg.replace(budget=b)) for b in budgets]
    orc.set_threads(4)
    for t in range(cfg.n_frames):
        frames, refs, outs, ref_outs = [], [], [], []
        for l in range(3):
            fi = gen.frame_inputs(cfg, t, layer=l)
            df = DeviceFrame(cfg, fi, "cuda")
            frames.append(df)
            ref_outs.append(oracles[l].attend(t, fi.q, fi.k, fi.v))
            refs.append(oracles[l].compress(fi.resid, fi.conf, fi.rho))
            outs.append(c.layer_attend(l, t, df.q, df.k, df.v))
        c.layers_compress(t, [f.resid for f in frames], frames[0].conf, frames[0].rho,
                          score_overrides=[torch.from_numpy(r["r"]).cuda() for r in refs])
        for l in range(3):
            err = np.abs(out_to_f32(outs[l]) - ref_outs[l])
            assert err.max() <= (ATT_F32 if dtype == gen.DTYPE_F32 else ATT_MAX), (t, l, err.max())
            sel = c.last_selection(l)
            np.testing.assert_array_equal(sel["survivors"], refs[l]["survivors"], err_msg=f"frame {t} layer {l}")
            fin = np.isfinite(refs[l]["r"])
            np.testing.assert_allclose(sel["r"][fin], refs[l]["r"][fin], rtol=0, atol=R_ATOL, err_msg=f"frame {t} layer {l}")
            st = c.stats(l)
            assert st["device_status"] == 0 and st["n_cached"] == oracles[l].n_rows == min((t + 1) * cfg.tokens_per_frame, budgets[l])
            assert st["anchor_frames"] == oracles[l].anchors() and st["evicted_total"] == oracles[l].evicted_total
            assert (st["n_protected_init"], st["n_protected_hist"]) == oracles[l].protected()
    for l in range(3):
        ex, rx = c.export(l), oracles[l].export()
        np.testing.assert_array_equal(ex["ids"], rx["ids"])
        np.testing.assert_array_equal(ex["flags"], rx["flags"])
        np.testing.assert_allclose(ex["stored"], rx["stored"], rtol=STORED_RTOL)
        assert np.array_equal(storage_to_f32(ex["k"], cfg.dtype), rx["k"])
        assert np.array_equal(storage_to_f32(ex["v"], cfg.dtype), rx["v"])
    # the call checks every layer before it changes anything
    f = frames[0]
    c.layer_attend(0, cfg.n_frames, f.q, f.k, f.v)           # only layer 0 has a pending frame now
    with pytest.raises(B.OvggtError) as e:
        c.layers_compress(cfg.n_frames, [f.resid] * 3, f.conf, f.rho)
    assert e.value.code == -4 and c.stats(0)["frames_seen"] == cfg.n_frames
    c.destroy()


def test_config2_full_size_through_layer_step_with_overlap():
    """The call the benchmark times: ovggt_layer_step on the benchmark configuration, where the compress half runs
    beside the attention on the handle's second stream.  Teacher-forced, so survivors and layout are bit-exact;
    the attention is checked on sampled rows while the compress half is running next to it."""
    cfg = gen.config_vggt_layer()
    orc.set_threads(max(1, min(32, torch.get_num_threads())))
    rows = np.sort(np.random.default_rng(12).choice(cfg.tokens_per_frame, 12, replace=False)).astype(np.int32)
    layer = orc.OracleLayer.from_stream(cfg)
    cache = B.OvggtCache.from_stream(cfg)
    for t in range(16):
        fi = gen.frame_inputs(cfg, t)
        df = DeviceFrame(cfg, fi, "cuda")
        check = t in (0, 12, 15)
        ref_out = layer.attend(t, fi.q, fi.k, fi.v, rows=rows, compute=check)
        ref = layer.compress(fi.resid, fi.conf, fi.rho)
        out = cache.layer_step(0, t, df.q, df.k, df.v, df.resid, df.conf, df.rho,
                               score_override=torch.from_numpy(ref["r"]).cuda())
        sel = cache.last_selection(0)
        np.testing.assert_array_equal(sel["survivors"], ref["survivors"], err_msg=f"frame {t}")
        fin = np.isfinite(ref["r"])
        np.testing.assert_allclose(sel["r"][fin], ref["r"][fin], rtol=0, atol=R_ATOL, err_msg=f"frame {t}")
        if check:
            err = np.abs(out_to_f32(out)[rows] - ref_out)
            assert err.max() <= ATT_MAX and err.mean() <= ATT_MEAN, (t, err.max(), err.mean())
    ex, rx = cache.export(0), layer.export()
    np.testing.assert_array_equal(ex["ids"], rx["ids"])
    np.testing.assert_array_equal(ex["flags"], rx["flags"])
    assert np.array_equal(storage_to_f32(ex["k"], cfg.dtype), rx["k"])
    assert np.array_equal(storage_to_f32(ex["v"], cfg.dtype), rx["v"])
    assert cache.stats(0)["device_status"] == 0
    cache.destroy()


def test_layer_step_at_steady_state_on_peaked_logits_every_key_block_matters():
    """ovggt_layer_step at the benchmark's steady state (N = B + M = 17758 rows, overlap on) with keys and values
    whose every 192-row block carries weight for some query rows (see attn_cases.tiled_hot_case): the cache is
    imported with the first B rows, the frame brings the last M, and the attention output is compared on rows of
    every group, rows of the ragged last query tile included."""
    cfg = gen.config_vggt_layer()
    orc.set_threads(max(1, min(32, torch.get_num_threads())))
    M, Bud, H = cfg.tokens_per_frame, cfg.budget, cfg.n_heads
    N = Bud + M
    q, k, v = tiled_hot_case(M, N, H, 47)
    rows = sampled_rows_all_groups(M, seed=9)
    cache = B.OvggtCache.from_stream(cfg)
    flags = np.zeros(Bud, np.uint8)
    flags[:M] = B.FLAG_INIT
    t_next = -(-Bud // M)
    cache.import_(0, np.arange(Bud, dtype=np.int64), flags, np.ones(Bud, np.float32), gen.bf16_round_bits(k[:Bud]),
                  gen.bf16_round_bits(v[:Bud]), next_frame_id=t_next, last_registration_frame=0)
    fi = gen.frame_inputs(cfg, t_next, fields=("resid",))
    to = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16).cuda()
    out = cache.layer_step(0, t_next, to(q), to(k[Bud:]), to(v[Bud:]), to(fi.resid), torch.from_numpy(fi.conf).cuda(), fi.rho)
    got = out_to_f32(out)
    assert np.isfinite(got).all()
    assert_attention_close_relative(got[rows], orc.attention(q, k, v, H, 64, rows=rows), "layer_step, steady state")
    st = cache.stats(0)
    assert st["device_status"] == 0 and st["n_cached"] == Bud and st["last_n_candidates"] == N
    cache.destroy()
