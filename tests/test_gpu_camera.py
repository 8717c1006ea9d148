"""The camera head's cache (Supp. C) through the C ABI against the CPU oracle: one token per frame, scored without
smoothing, its anchor flags mirrored from an aggregator handle that runs the same stream."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2603_05959_b200 import binding as B
from paper_2603_05959_b200 import inputs as gen
from paper_2603_05959_b200.stream import DeviceFrame, out_to_f32, storage_to_f32

pytestmark = pytest.mark.gpu

R_ATOL = 2e-5
ATT_MAX, ATT_MEAN, ATT_F32 = 2e-2, 2e-3, 1e-4


def camera_token(cfg, t, tag):
    """One seeded row of cfg.dim values for frame t: the camera token's q, k, v (tags 1-3) or residual (tag 4)."""
    rng = np.random.Generator(np.random.Philox(key=[np.uint64(cfg.seed + 77), np.uint64((t << 8) | tag)]))
    return gen.round_to_dtype(rng.standard_normal((1, cfg.dim), dtype=np.float32) * (1.0 + 0.1 * tag), cfg.dtype)


def dev(x, dtype):
    return torch.from_numpy(np.ascontiguousarray(x)).to(B.torch_dtype(dtype)).cuda()


@pytest.mark.parametrize("dtype,score_mode", [(gen.DTYPE_F32, gen.SCORE_HYBRID), (gen.DTYPE_BF16, gen.SCORE_HYBRID),
                                              (gen.DTYPE_F32, gen.SCORE_RESIDUAL_STORED)])
def test_camera_cache_mirrors_the_aggregator_and_matches_the_oracle(dtype, score_mode):
    cfg = gen.config_tiny().replace(tau=0.95, min_anchor_interval=2, k_max=2, n_frames=24, dtype=dtype)
    cam_budget = 6
    orc.set_threads(4)
    agg, agg_o = B.OvggtCache.from_stream(cfg), orc.OracleLayer.from_stream(cfg)
    cam = B.OvggtCache.camera(n_heads=cfg.n_heads, budget=cam_budget, k_max=cfg.k_max, dtype=dtype, score_mode=score_mode)
    cam_o = orc.OracleLayer.camera(n_heads=cfg.n_heads, head_dim=64, budget=cam_budget, k_max=cfg.k_max,
                                   score_mode=score_mode)
    with pytest.raises(B.OvggtError):
        agg.anchor_decision(0)                              # nothing decided yet
    demotions = 0
    for t in range(cfg.n_frames):
        # the aggregator's step, teacher-forced so that both sides keep the same cache
        fi = gen.frame_inputs(cfg, t)
        df = DeviceFrame(cfg, fi, "cuda")
        agg_o.attend(t, fi.q, fi.k, fi.v, compute=False)
        dec = agg_o.compress(fi.resid, fi.conf, fi.rho)
        agg.layer_step(0, t, df.q, df.k, df.v, df.resid, df.conf, df.rho, score_override=torch.from_numpy(dec["r"]).cuda())
        reg, dem = agg.anchor_decision(t)
        assert (reg, dem) == (dec["registered"], dec["demoted_frame"]), t
        demotions += dem >= 0
        # the camera head's step on its own token
        q, k, v, r = (camera_token(cfg, t, tag) for tag in (1, 2, 3, 4))
        ref_out = cam_o.attend(t, q, k, v)
        ref = cam_o.compress_camera(r, dec["registered"], dec["demoted_frame"])
        out = cam.layer_attend(0, t, dev(q, dtype), dev(k, dtype), dev(v, dtype))
        cam.camera_compress(0, t, dev(r, dtype), reg, dem, score_override=torch.from_numpy(ref["r"]).cuda())
        err = np.abs(out_to_f32(out) - ref_out)
        if dtype == gen.DTYPE_F32:
            assert err.max() <= ATT_F32, (t, err.max())
        else:
            assert err.max() <= ATT_MAX and err.mean() <= ATT_MEAN, (t, err.max(), err.mean())
        sel = cam.last_selection(0)
        np.testing.assert_array_equal(sel["survivors"], ref["survivors"], err_msg=f"frame {t}")
        fin = np.isfinite(ref["r"])
        assert np.array_equal(np.isinf(sel["r"]), ~fin), t
        tol = dict(rtol=0, atol=R_ATOL) if score_mode == gen.SCORE_HYBRID else dict(rtol=2e-5, atol=0)
        np.testing.assert_allclose(sel["r"][fin], ref["r"][fin], err_msg=f"frame {t}", **tol)
        st = cam.stats(0)
        assert st["device_status"] == 0 and st["n_cached"] == min(t + 1, cam_budget)
        assert st["anchor_frames"] == agg_o.anchors() == cam_o.anchors()
        assert st["n_protected_init"] == 1 and st["n_protected_hist"] == len(agg_o.anchors())
        ex, rx = cam.export(0), cam_o.export()
        np.testing.assert_array_equal(ex["ids"], rx["ids"])
        np.testing.assert_array_equal(ex["flags"], rx["flags"])
        np.testing.assert_allclose(ex["stored"], rx["stored"], rtol=2e-5)       # the raw norm: no smoothing
        assert np.array_equal(storage_to_f32(ex["k"], dtype), rx["k"])
        assert np.array_equal(storage_to_f32(ex["v"], dtype), rx["v"])
    assert demotions >= 2 and cam_o.evicted_total > 0
    agg.destroy(); cam.destroy()


def test_camera_cache_call_rules():
    cfg = gen.config_tiny()
    cam = B.OvggtCache.camera(n_heads=cfg.n_heads, budget=5, dtype=gen.DTYPE_F32)
    agg = B.OvggtCache.from_stream(cfg)
    x = torch.zeros((1, cfg.dim), device="cuda")
    with pytest.raises(B.OvggtError) as e:                  # a camera cache cannot decide anchors by itself
        cam.layer_step(0, 0, x, x, x, x)
    assert e.value.code == -1
    cam.layer_attend(0, 0, x, x, x)
    with pytest.raises(B.OvggtError):
        cam.layer_compress(0, 0, x)
    cam.camera_compress(0, 0, x, False, -1)
    f = DeviceFrame(cfg, gen.frame_inputs(cfg, 0), "cuda")
    agg.layer_attend(0, 0, f.q, f.k, f.v)
    with pytest.raises(B.OvggtError) as e:                  # and an aggregator cache takes no mirrored decision
        agg.camera_compress(0, 0, f.resid, False, -1)
    assert e.value.code == -1
    with pytest.raises(B.OvggtError):                       # 1 + K_max tokens must fit
        B.OvggtCache.camera(n_heads=4, budget=3, k_max=3)
    cam.destroy(); agg.destroy()
