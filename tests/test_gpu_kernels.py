"""GPU parity of each kernel against the CPU oracle, through the C ABI (binding -> libovggt.so)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2603_05959_b200 import binding as B
from paper_2603_05959_b200 import inputs as gen

from attn_cases import assert_attention_close_relative, sampled_rows_all_groups, tiled_hot_case

pytestmark = pytest.mark.gpu

# Tolerances (derived from the arithmetic):
#  fp32 fixed-order sums of <= 1024 squares against fp64: relative 1e-5
#  d = 1 - cos with an fp32 column sum over up to ~32K rows: absolute 5e-6
#  bf16 attention against the fp64 oracle: max-abs 2e-2, mean-abs 2e-3; fp32 attention: 1e-4
NORM_RTOL = 1e-5
DIV_ATOL = 5e-6
ATT_MAX, ATT_MEAN, ATT_F32 = 2e-2, 2e-3, 1e-4


def dev(x, dtype):
    t = torch.from_numpy(np.ascontiguousarray(x))
    return t.to(torch.bfloat16 if dtype == gen.DTYPE_BF16 else torch.float32).cuda()


def rnd(shape, dtype, seed, scale=1.0):
    x = np.random.default_rng(seed).standard_normal(shape).astype(np.float32) * np.float32(scale)
    return gen.round_to_dtype(x, dtype)


@pytest.mark.parametrize("rows,C,dtype", [(1374, 1024, 1), (69, 256, 0), (7, 64, 1), (1, 64, 0), (333, 768, 1),
                                          (100, 1024, 0)])
def test_row_norms(rows, C, dtype):
    x = rnd((rows, C), dtype, 1) * np.exp(np.random.default_rng(2).normal(0, 0.75, (rows, 1))).astype(np.float32)
    x = gen.round_to_dtype(x, dtype)
    got = B.k_row_norms(dev(x, dtype)).cpu().numpy()
    np.testing.assert_allclose(got, orc.residual_norms(x), rtol=NORM_RTOL)


def test_row_norms_is_deterministic_and_handles_zero_rows():
    x = dev(rnd((500, 1024), 1, 3), 1)
    a, b = B.k_row_norms(x), B.k_row_norms(x)
    assert torch.equal(a, b)
    z = torch.zeros((4, 256), dtype=torch.float32, device="cuda")
    assert torch.equal(B.k_row_norms(z), torch.zeros(4, device="cuda"))
    assert B.k_row_norms(torch.empty((0, 256), dtype=torch.float32, device="cuda")).numel() == 0


@pytest.mark.parametrize("rows,C,dtype", [(3000, 1024, 1), (325, 256, 0), (1, 64, 1), (17, 128, 0), (16384, 1024, 1)])
def test_diversity(rows, C, dtype):
    K = rnd((rows, C), dtype, 4) + np.float32(0.25)      # a non-zero centroid
    K = gen.round_to_dtype(K, dtype)
    got = B.k_diversity(dev(K, dtype)).cpu().numpy()
    np.testing.assert_allclose(got, orc.diversity(K), rtol=0, atol=DIV_ATOL)


def test_diversity_degenerate_rows():
    K = np.zeros((5, 64), np.float32)
    K[0, 0] = 1.0; K[1, 0] = 2.0; K[2, 0] = -1.0; K[4, 1] = 3.0
    got = B.k_diversity(dev(K, 0)).cpu().numpy()
    np.testing.assert_allclose(got, orc.diversity(K), atol=DIV_ATOL)
    assert got[3] == 1.0                                  # a zero key: cosine 0 by convention


def _select_case(N, seed, levels=None, specials=True, p_prot=0.1):
    rng = np.random.default_rng(seed)
    r = rng.random(N).astype(np.float32) if levels is None else \
        (rng.integers(0, levels, N).astype(np.float32) / np.float32(levels))
    if specials and N > 8:
        r[rng.integers(0, N, 4)] = [np.nan, -np.inf, np.inf, -0.0]
    flags = (rng.random(N) < p_prot).astype(np.uint8) * rng.integers(1, 3, N).astype(np.uint8)
    return r, flags


@pytest.mark.parametrize("N", [5, 325, 1500, 17758, 34142, 70001])
@pytest.mark.parametrize("levels", [None, 3])
def test_select_bit_exact(N, levels):
    r, flags = _select_case(N, N + (levels or 0), levels)
    P = int(np.count_nonzero(flags))
    for Bud in sorted({P, P + 1, (P + N) // 2, N - 1, N, N + 5}):
        got = B.k_select(torch.from_numpy(r).cuda(), torch.from_numpy(flags).cuda(), Bud).cpu().numpy()
        np.testing.assert_array_equal(got, orc.select(r, flags, Bud))


def test_select_batched_and_all_equal():
    N, Bud, batch = 4000, 1500, 5
    rs, fs = zip(*[_select_case(N, 50 + b, 4 if b % 2 else None) for b in range(batch)])
    r = np.stack(rs); f = np.stack(fs)
    r[4] = 0.25                                           # every priority equal: pure position order
    got = B.k_select(torch.from_numpy(r).cuda(), torch.from_numpy(f).cuda(), Bud).cpu().numpy()
    for b in range(batch):
        np.testing.assert_array_equal(got[b], orc.select(r[b], f[b], Bud))


@pytest.mark.parametrize("C,dtype", [(1024, 1), (256, 0), (64, 1)])
def test_compact_is_exact_gather(C, dtype):
    rng = np.random.default_rng(7)
    N = 3001
    k, v = rnd((N, C), dtype, 8), rnd((N, C), dtype, 9)
    surv = np.sort(rng.choice(N, 1777, replace=False)).astype(np.int32)
    kd, vd = B.k_compact(dev(k, dtype), dev(v, dtype), torch.from_numpy(surv).cuda())
    assert np.array_equal(kd.float().cpu().numpy(), k[surv]) and np.array_equal(vd.float().cpu().numpy(), v[surv])
    kd, vd = B.k_compact(dev(k, dtype), dev(v, dtype), torch.empty(0, dtype=torch.int32, device="cuda"))
    assert kd.shape[0] == 0


BOTH_REFERENCES = pytest.mark.parametrize("bounded", [False, True], ids=["tracked-max", "key-bound"])


def _attn_check(M, N, H, dtype, seed, rows=None, qscale=1.0, bounded=False):
    q, k, v = rnd((M, H * 64), dtype, seed, qscale), rnd((N, H * 64), dtype, seed + 1), rnd((N, H * 64), dtype, seed + 2)
    got = B.k_attention(dev(q, dtype), dev(k, dtype), dev(v, dtype), H, bounded=bounded).float().cpu().numpy()
    assert np.isfinite(got).all()
    ref = orc.attention(q, k, v, H, 64, rows=rows)
    g = got if rows is None else got[rows]
    err = np.abs(g - ref)
    if dtype == gen.DTYPE_F32:
        assert err.max() <= ATT_F32
    else:
        assert err.max() <= ATT_MAX and err.mean() <= ATT_MEAN, (err.max(), err.mean())
    return got


@pytest.mark.parametrize("M,N,H", [(128, 128, 1), (1, 1, 1), (94, 129, 2), (200, 1000, 2), (69, 325, 4),
                                   (300, 4096, 3), (129, 2500, 1)])
@BOTH_REFERENCES
def test_attention_bf16_small(M, N, H, bounded):
    orc.set_threads(8)
    _attn_check(M, N, H, gen.DTYPE_BF16, 10 + M + N, bounded=bounded)


@BOTH_REFERENCES
def test_attention_bf16_large_logits_exercise_rescaling(bounded):
    orc.set_threads(8)
    _attn_check(150, 1500, 2, gen.DTYPE_BF16, 77, qscale=6.0, bounded=bounded)


def test_key_norm_bound_is_the_largest_per_head_key_norm():
    k = rnd((3001, 5 * 64), gen.DTYPE_BF16, 3) * np.linspace(0.5, 2.0, 5, dtype=np.float32).repeat(64)[None, :]
    k = gen.round_to_dtype(k, gen.DTYPE_BF16)
    got = B.k_key_norm_bound(dev(k, 1), 5).cpu().numpy()
    want = (k.astype(np.float64).reshape(3001, 5, 64) ** 2).sum(-1).max(0)
    np.testing.assert_allclose(got, want, rtol=1e-5)
    assert B.k_key_norm_bound(torch.empty((0, 128), dtype=torch.bfloat16, device="cuda"), 2).tolist() == [0.0, 0.0]


@BOTH_REFERENCES
def test_attention_bf16_scores_rising_along_the_keys(bounded):
    """Keys ordered so that every score half outgrows the running reference maximum by far more than the lazy
    threshold: each round takes the rescale-and-recompute path, and the softmax concentrates on the last keys.
    (With the key-norm bound on, that bound lies hundreds of powers of two above the first scores, which the kernel
    must notice and fall back to tracking the maximum.)"""
    orc.set_threads(8)
    M, N, H, dt = 140, 1100, 2, gen.DTYPE_BF16
    rng = np.random.default_rng(91)
    u = rng.standard_normal(64).astype(np.float32)
    u /= np.linalg.norm(u)
    ramp = (np.arange(N, dtype=np.float32) * 0.25)[:, None]                  # +24 (natural-log units / 8 * 8) per 96 keys
    k = np.concatenate([ramp * u[None, :] + 0.1 * rng.standard_normal((N, 64)).astype(np.float32) for _ in range(H)], axis=1)
    q = np.concatenate([(8.0 + rng.random((M, 1)).astype(np.float32)) * u[None, :] for _ in range(H)], axis=1)
    v = rng.standard_normal((N, H * 64)).astype(np.float32)
    q, k, v = (gen.round_to_dtype(x, dt) for x in (q, k, v))
    got = B.k_attention(dev(q, dt), dev(k, dt), dev(v, dt), H, bounded=bounded).float().cpu().numpy()
    ref = orc.attention(q, k, v, H, 64)
    err = np.abs(got - ref)
    assert np.isfinite(got).all() and err.max() <= ATT_MAX and err.mean() <= ATT_MEAN, (err.max(), err.mean())


@pytest.mark.parametrize("M,N,H", [(69, 325, 4), (1, 1, 1), (130, 700, 2)])
def test_attention_fp32(M, N, H):
    orc.set_threads(8)
    _attn_check(M, N, H, gen.DTYPE_F32, 20 + M)


@BOTH_REFERENCES
def test_attention_bf16_full_size_sampled_rows(bounded):
    """The bench configuration: 1374 queries x 17758 keys x 16 heads; the oracle checks sampled rows."""
    orc.set_threads(max(1, min(32, torch.get_num_threads())))
    rows = np.sort(np.random.default_rng(5).choice(1374, 24, replace=False)).astype(np.int32)
    rows[0], rows[-1] = 0, 1373
    got = _attn_check(1374, 17758, 16, gen.DTYPE_BF16, 30, rows=rows, bounded=bounded)
    # properties that hold at any size: finite, and each output inside the range of V per column
    assert np.abs(got).max() < 6.0


@BOTH_REFERENCES
def test_attention_bf16_full_size_peaked_logits_every_key_block_matters(bounded):
    """The bench shape again (5 KV splits x 19 tiles, 94-row tail, ragged last query tile) on data that can fail it:
    see tiled_hot_case.  As a self-check of the data, the reference is recomputed without the last key block and
    without the middle fifth of the keys and must then violate the criterion the kernel has to meet."""
    orc.set_threads(max(1, min(32, torch.get_num_threads())))
    M, N, H = 1374, 17758, 16
    q, k, v = tiled_hot_case(M, N, H, 41)
    rows = sampled_rows_all_groups(M)
    assert len(rows) >= 24 and rows.max() >= 1280
    got = B.k_attention(dev(q, 1), dev(k, 1), dev(v, 1), H, bounded=bounded).float().cpu().numpy()
    assert np.isfinite(got).all()
    ref = orc.attention(q, k, v, H, 64, rows=rows)
    assert_attention_close_relative(got[rows], ref, "bench shape, peaked")
    for lo, hi in ((92 * 192, N), (7104, 10752)):            # the ragged last block; KV tiles 37..55 (the middle split)
        keep = np.r_[0:lo, hi:N]
        broken = orc.attention(q, k[keep], v[keep], H, 64, rows=rows)
        with pytest.raises(AssertionError):
            assert_attention_close_relative(broken, ref)


@BOTH_REFERENCES
@pytest.mark.parametrize("M,N,H", [(300, 2500, 2), (1041, 13329, 2)])
def test_attention_bf16_peaked_logits_other_shapes(M, N, H, bounded):
    orc.set_threads(max(1, min(32, torch.get_num_threads())))
    q, k, v = tiled_hot_case(M, N, H, 43 + M)
    rows = sampled_rows_all_groups(M)
    got = B.k_attention(dev(q, 1), dev(k, 1), dev(v, 1), H, bounded=bounded).float().cpu().numpy()
    assert_attention_close_relative(got[rows], orc.attention(q, k, v, H, 64, rows=rows), f"{M}x{N}")


@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (5, 8, 64), (130, 136, 192), (1374, 3072, 1024), (1041, 1024, 4096)])
def test_gemm_bf16_against_the_plain_product(M, N, K):
    """The scaffold GEMM (not a step of the paper's path): C = A B against the definition in fp64 (numpy's matmul on
    the same bf16-rounded inputs); bf16 output: half an ulp of the result plus fp32 accumulation error."""
    a, b = rnd((M, K), gen.DTYPE_BF16, 3 + M), rnd((K, N), gen.DTYPE_BF16, 4 + N, scale=0.05)
    got = B.k_gemm_bf16(dev(a, 1), dev(b, 1)).float().cpu().numpy()
    ref = a.astype(np.float64) @ b.astype(np.float64)
    np.testing.assert_allclose(got, ref, rtol=2 ** -8, atol=1e-3 * np.abs(ref).max())
    with pytest.raises(B.OvggtError) as e:                    # K must be a multiple of 64
        B.k_gemm_bf16(dev(a[:, :K - 8], 1), dev(b[:K - 8], 1))
    assert e.value.code == -10


def test_attention_is_deterministic():
    q, k, v = (dev(rnd(s, 1, i), 1) for i, s in enumerate(((500, 256), (3000, 256), (3000, 256))))
    a, b = B.k_attention(q, k, v, 4), B.k_attention(q, k, v, 4)
    assert torch.equal(a, b)
