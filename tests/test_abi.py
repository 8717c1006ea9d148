"""CPU checks of the C-ABI library: it loads, exports every symbol the header declares, and its
host-side validation answers with the documented error codes before touching a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2603_05959_b200 import binding as B
from paper_2603_05959_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B.lib()


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(ovggt_\w+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"
    assert set(B.EXPORTED) == names


def _cfg(**over):
    kw = dict(n_layers=1, n_heads=4, head_dim=64, n_special=5, grid_h=8, grid_w=8, budget=256,
              anchor_tokens=8, k_max=3, min_anchor_interval=4, tau=0.2, alpha=0.5, beta=0.5,
              protect_first_frame=1, score_mode=0, dtype=0, compaction=1, random_seed=0, camera_head=0)
    kw.update(over)
    budgets = (C.c_int32 * kw["n_layers"])(*([kw.pop("budget")] * kw["n_layers"]))
    cfg = B.OvggtConfig(kw["n_layers"], kw["n_heads"], kw["head_dim"], kw["n_special"], kw["grid_h"],
                        kw["grid_w"], budgets, kw["anchor_tokens"], kw["k_max"], kw["min_anchor_interval"],
                        kw["tau"], kw["alpha"], kw["beta"], kw["protect_first_frame"], kw["score_mode"],
                        kw["dtype"], kw["compaction"], kw["random_seed"], kw["camera_head"], None, 0)
    cfg._keep = budgets
    return cfg


def test_workspace_bytes_is_a_pure_host_function(lib):
    cfg = _cfg()
    need = lib.ovggt_workspace_bytes(C.byref(cfg))
    M, Cdim, R = 69, 256, 256 + 69
    assert need >= 4 * R * Cdim * 4              # stable gather: two K and two V buffers of B + M rows, fp32
    holes = lib.ovggt_workspace_bytes(C.byref(_cfg(compaction=0)))
    assert 2 * R * Cdim * 4 <= holes < need      # hole filling: one K and one V buffer
    big = lib.ovggt_workspace_bytes(C.byref(_cfg(budget=512)))
    assert big > need
    # the bf16 VGGT-shaped layer: 2 x 2 x (16384 + 1374) x 1024 x 2 bytes of K/V
    need2 = lib.ovggt_workspace_bytes(C.byref(_cfg(n_heads=16, grid_h=37, grid_w=37, budget=16384,
                                                    anchor_tokens=64, dtype=1)))
    assert need2 >= 4 * 17758 * 1024 * 2 and need2 < 3 * 4 * 17758 * 1024 * 2


def test_create_reports_config_errors_without_a_gpu(lib):
    h = C.c_void_p()
    bad = [(_cfg(head_dim=32), -1), (_cfg(n_layers=0, budget=256), -1), (_cfg(dtype=7), -1),
           (_cfg(alpha=1.5), -1), (_cfg(k_max=17), -1), (_cfg(anchor_tokens=65), -1), (_cfg(compaction=2), -1), (_cfg(score_mode=5), -1),
           (_cfg(camera_head=1, n_special=1, grid_h=0, grid_w=0, anchor_tokens=0, budget=8, score_mode=3), -1),
           (_cfg(camera_head=1), -1), (_cfg(camera_head=1, n_special=1, grid_h=0, grid_w=0, anchor_tokens=0, budget=3), -3),
           (_cfg(budget=68), -3), (_cfg(budget=69 + 3 * 8 - 1), -3)]
    for cfg, code in bad:
        assert lib.ovggt_workspace_bytes(C.byref(cfg)) == 0
        assert lib.ovggt_cache_create(C.byref(cfg), C.byref(h)) == code
        assert not h.value
    # a budget whose B + M candidates do not fit the selection cluster's shared memory is refused at create,
    # not at the first step
    huge = _cfg(n_heads=16, grid_h=37, grid_w=37, budget=120000, anchor_tokens=64, dtype=1)
    assert lib.ovggt_workspace_bytes(C.byref(huge)) == 0
    assert lib.ovggt_cache_create(C.byref(huge), C.byref(h)) == -10 and not h.value
    assert lib.ovggt_workspace_bytes(C.byref(_cfg(n_heads=16, grid_h=37, grid_w=37, budget=65536, anchor_tokens=64,
                                                  dtype=1))) > 0
    cam = _cfg(camera_head=1, n_special=1, grid_h=0, grid_w=0, anchor_tokens=0, budget=4)   # 1 + K_max tokens
    assert lib.ovggt_workspace_bytes(C.byref(cam)) > 0
    ok = _cfg(budget=69 + 3 * 8)
    assert lib.ovggt_workspace_bytes(C.byref(ok)) > 0
    assert lib.ovggt_cache_create(C.byref(ok), C.byref(h)) == -1          # no workspace given
    ok.workspace, ok.workspace_bytes = 1024 + 16, 1 << 40
    assert lib.ovggt_cache_create(C.byref(ok), C.byref(h)) == -5          # misaligned workspace
    ok.workspace, ok.workspace_bytes = 4096, 1024
    assert lib.ovggt_cache_create(C.byref(ok), C.byref(h)) == -6          # workspace too small
    assert lib.ovggt_cache_create(None, C.byref(h)) == -1
    assert lib.ovggt_cache_destroy(None) == -1


def test_null_handle_and_strerror(lib):
    io = B.OvggtFrameIO()
    for name in ("ovggt_layer_attend", "ovggt_layer_compress", "ovggt_layer_step", "ovggt_layer_step_host"):
        assert getattr(lib, name)(None, 0, C.byref(io), None) == -1
    st = B.OvggtStats()
    assert lib.ovggt_cache_stats(None, 0, C.byref(st)) == -1
    assert lib.ovggt_cache_reset(None) == -1
    seen = {lib.ovggt_strerror(c) for c in range(0, -11, -1)}
    assert len(seen) == 11 and b"unknown error" not in seen
    assert lib.ovggt_strerror(-99) == b"unknown error"
    assert lib.ovggt_kernel_launches() == 0
    assert lib.ovggt_k_row_norms(None, 1, 64, 0, None, None) == -1
    assert lib.ovggt_k_select(None, None, 0, 0, 1, None, None, None) == -1
    assert lib.ovggt_k_gemm_bf16(None, None, 1, 8, 64, None, None, None) == -1


def test_checked_build_compiles_and_exports_the_same_symbols():
    """The variant with range-checked indices (-DOVGGT_BOUNDS_CHECK) is the same library: it must build for sm_100a
    and export every declared symbol."""
    path = build_mod.build(checked=True)
    assert path.endswith("libovggt_checked.so") and os.path.exists(path)
    checked = C.CDLL(path)
    for n in declared_symbols():
        assert hasattr(checked, n), n


def test_build_refuses_an_attention_kernel_with_another_launch_register_count():
    """setmaxnreg moves registers inside the pool the CTA is launched with; the build checks ptxas' launch count
    against the count the warpgroup budgets in the source were written for."""
    import re
    from paper_2603_05959_b200 import build as bld
    src = open(os.path.join(bld.CSRC, "attn_tcgen05.cuh")).read()
    want = int(re.search(r"constexpr int kRegsLaunch = (\d+);", src).group(1))
    soft = int(re.search(r"constexpr int kRegsSoftmax = (\d+), kRegsOther = (\d+);", src).group(1))
    other = int(re.search(r"constexpr int kRegsSoftmax = (\d+), kRegsOther = (\d+);", src).group(2))
    threads = int(re.search(r"constexpr int kAttnThreads = (\d+);", src).group(1))
    assert threads == 256 and 128 * soft + 128 * other <= threads * want        # the pool rule itself
    log = ("ptxas info    : Compiling entry function '_ZN5ovggt14k_attn_tcgen05E14CUtensorMap_stS0_S0_NS_10AttnParamsE' "
           "for 'sm_100a'\nptxas info    : Function properties\nptxas info    : Used %d registers, used 1 barriers\n")
    bld.check_register_pool(log % want)
    with pytest.raises(RuntimeError):
        bld.check_register_pool(log % (want - 8))
    with pytest.raises(RuntimeError):
        bld.check_register_pool("ptxas info    : nothing about that kernel\n")
