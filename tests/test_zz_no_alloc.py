"""ovggt_k_diversity_static: the allocation-free variant of the key-diversity kernel.

Some users of the library cannot give it scratch memory: their process has already handed the GPU's
memory to an allocator of its own, or they sit in a per-frame loop where a driver allocation would stall
the device.  For them the library carries its scratch inside itself.  This test calls the variant through
the C ABI twice in a row (a large problem first, then a smaller one that leaves stale values behind it in
the shared array) and requires the same numbers the ordinary entry point gives, and both against the CPU
oracle's definition of the score, so that the two entry points cannot be wrong together.  It is collected
last so that a failure here cannot hide a failure elsewhere."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2603_05959_b200 import binding as B
from paper_2603_05959_b200 import inputs as gen

pytestmark = pytest.mark.gpu

DIV_ATOL = 5e-6      # the tolerance of the diversity parity tests


def _keys(rows, C, dtype, seed):
    """(device tensor in the storage type, the same values as float32 on the host for the oracle)"""
    x = np.random.default_rng(seed).standard_normal((rows, C)).astype(np.float32) + np.float32(0.25)
    x = gen.round_to_dtype(x, dtype)
    t = torch.from_numpy(x)
    return t.to(torch.bfloat16 if dtype == gen.DTYPE_BF16 else torch.float32).cuda(), x


def test_static_scratch_variant_matches_on_two_calls_in_a_row():
    orc.set_threads(8)
    big, big_host = _keys(16384, 1024, gen.DTYPE_BF16, 1)
    small, small_host = _keys(700, 256, gen.DTYPE_F32, 2)
    ref_big, ref_small = B.k_diversity(big), B.k_diversity(small)
    orc_big, orc_small = orc.diversity(big_host), orc.diversity(small_host)
    d_big = torch.full((16384,), -7.0, dtype=torch.float32, device="cuda")
    d_small = torch.full((700,), -7.0, dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    B.k_diversity_static(big, d_big)
    B.k_diversity_static(small, d_small)        # same stream: ordered after the first, reuses its scratch
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    np.testing.assert_allclose(d_big.cpu().numpy(), ref_big.cpu().numpy(), rtol=0, atol=DIV_ATOL)
    np.testing.assert_allclose(d_small.cpu().numpy(), ref_small.cpu().numpy(), rtol=0, atol=DIV_ATOL)
    np.testing.assert_allclose(d_big.cpu().numpy(), orc_big, rtol=0, atol=DIV_ATOL)
    np.testing.assert_allclose(d_small.cpu().numpy(), orc_small, rtol=0, atol=DIV_ATOL)
    # and once more with the first problem: the array now holds the small problem's leftovers
    d_again = torch.empty_like(d_big)
    B.k_diversity_static(big, d_again)
    torch.cuda.synchronize()
    np.testing.assert_allclose(d_again.cpu().numpy(), ref_big.cpu().numpy(), rtol=0, atol=DIV_ATOL)
    np.testing.assert_allclose(d_again.cpu().numpy(), orc_big, rtol=0, atol=DIV_ATOL)


def test_static_scratch_variant_rejects_sizes_beyond_its_capacity():
    K = torch.zeros((8, 2048), dtype=torch.bfloat16, device="cuda")
    d = torch.full((8,), 3.0, dtype=torch.float32, device="cuda")
    with pytest.raises(B.OvggtError) as e:
        B.k_diversity_static(K, d)
    assert e.value.code == -11 and "capacity" in str(e.value)
    torch.cuda.synchronize()
    assert torch.all(d == 3.0)                   # nothing was launched
