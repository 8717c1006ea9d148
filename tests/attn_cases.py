"""Attention inputs that can fail a kernel at the benchmark's shape, shared by the GPU parity tests.

Holds no arithmetic of the method: it only builds q, k, v arrays and compares two outputs."""
import numpy as np

from paper_2603_05959_b200 import inputs as gen

ATT_MAX, ATT_MEAN = 2e-2, 2e-3          # the bf16 attention tolerances (max-abs, mean-abs)


def tiled_hot_case(M, N, H, seed, groups=12, tile=192, gain=8.0):
    """Peaked attention whose mass is spread over the whole key range in a known pattern.  The keys of 192-row
    block b point along direction u[b % groups], query row m along u[m % groups], so a query puts nearly all of its
    weight on every groups-th block of keys - first block to last, ragged tail included - and the values of a block
    share one random vector.  Leaving out any one block, or a whole range of them, moves the output of the rows
    that attend to it by tens of percent of its size, far outside any rounding tolerance."""
    rng = np.random.default_rng(seed)
    u = np.linalg.qr(rng.standard_normal((64, groups)))[0].T.astype(np.float32)          # [groups, 64] orthonormal
    blk = np.arange(N) // tile
    nblk = int(blk.max()) + 1
    k = np.concatenate([gain * u[blk % groups] + 0.5 * rng.standard_normal((N, 64)).astype(np.float32)
                        for _ in range(H)], axis=1)
    q = np.concatenate([gain * u[np.arange(M) % groups] + 0.5 * rng.standard_normal((M, 64)).astype(np.float32)
                        for _ in range(H)], axis=1)
    w = rng.standard_normal((nblk, H * 64)).astype(np.float32)
    v = w[blk] + 0.25 * rng.standard_normal((N, H * 64)).astype(np.float32)
    return (gen.round_to_dtype(x, gen.DTYPE_BF16) for x in (q, k, v))


def assert_attention_close_relative(got, ref, what=""):
    """The absolute tolerances of the bf16 path, and each row within 5 % of that row's largest reference entry."""
    err = np.abs(got - ref)
    assert err.max() <= ATT_MAX and err.mean() <= ATT_MEAN, (what, err.max(), err.mean())
    scale = np.abs(ref).max(axis=1)
    assert np.all(err.max(axis=1) <= 0.05 * scale), (what, float((err.max(axis=1) / scale).max()))


def sampled_rows_all_groups(M, groups=12, seed=5):
    """Two query rows of every group, rows of the first and of the last (ragged) 128-row query tile among them."""
    rng = np.random.default_rng(seed)
    last_tile = (M - 1) // 128 * 128
    rows = set()
    for g in range(groups):
        cand = np.arange(g, M, groups)
        rows.add(int(rng.choice(cand[cand < last_tile])))
        rows.add(int(rng.choice(cand[cand >= last_tile])))
    return np.array(sorted(rows), dtype=np.int32)
