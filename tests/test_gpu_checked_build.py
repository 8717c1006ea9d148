"""The parity cases with small and ragged shapes once more against the library built with range-checked indices
(-DOVGGT_BOUNDS_CHECK): every index a kernel reads from device memory - survivor lists, slots, move lists - is tested
against its range before it is used, and a violation would show up as a non-zero device status, which these tests
assert to be zero after every frame.  Runs in a child process because the library is chosen when it is loaded."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CASES = ("test_config1_tiny_fp32_every_frame or test_bf16_ragged_midsize_stream or test_budget_not_a_multiple "
         "or test_stored_residual_mode_and_no_anchors or test_random_eviction_mode or test_all_layers_compressed "
         "or test_config1_frequent_anchors or test_multi_layer_handle")


def test_small_and_ragged_parity_cases_under_the_checked_build():
    from paper_2603_05959_b200 import build as build_mod
    build_mod.build(checked=True)
    env = dict(os.environ, OVGGT_LIBRARY="checked")
    probe = subprocess.run([sys.executable, "-c", "from paper_2603_05959_b200 import binding as B; print(B.LIB_PATH)"],
                           cwd=ROOT, env=env, capture_output=True, text=True, timeout=120)
    assert probe.stdout.strip().endswith("libovggt_checked.so"), probe.stdout + probe.stderr
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_stream.py"),
                        os.path.join(ROOT, "tests", "test_gpu_camera.py"), "-m", "gpu", "-q", "-x", "-k",
                        CASES + " or camera"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-1000:]
    assert " passed" in r.stdout and "failed" not in r.stdout
