"""Do the GPU parity tests notice a wrong oracle?  The mistake is planted in a compiled COPY of the oracle (on the
CPU); the named GPU parity test is then run against that copy in a child process and has to fail: the library, which
is right, no longer agrees with it.  (The counterpart for the oracle's own pins is tests/test_oracle_mutants.py.)"""
import os
import subprocess
import sys

import pytest

from oracle import build as oracle_build
from test_oracle_mutants import MISTAKES

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BY_NAME = {m[0]: m for m in MISTAKES}

CASES = [
    ("Eq. 5 without the square root", "tests/test_gpu_kernels.py", "test_row_norms"),
    # (alpha = beta = 0.5 in the default configuration, where these two swaps change nothing: a case with other values)
    ("Eq. 6 with alpha and 1 - alpha swapped", "tests/test_gpu_stream.py", "test_stored_residual_mode_and_no_anchors"),
    ("diversity as the cosine itself", "tests/test_gpu_kernels.py", "test_diversity"),
    ("Eq. 7 with the two weights swapped", "tests/test_gpu_stream.py", "test_stored_residual_mode_and_no_anchors"),
    ("Eq. 8 with ties going to the higher position", "tests/test_gpu_kernels.py", "test_select_bit_exact"),
    ("Eq. 6 with rows and columns of the map swapped", "tests/test_gpu_stream.py", "test_config1_tiny_fp32_every_frame"),
    ("FIFO that drops the newest anchor", "tests/test_gpu_stream.py", "test_config1_frequent_anchors_exercise_fifo_demotion"),
    ("attention without 1 / sqrt(d)", "tests/test_gpu_kernels.py", "test_attention_bf16_small"),
    ("anchor tokens flagged without the offset of the special tokens", "tests/test_gpu_stream.py",
     "test_config1_frequent_anchors_exercise_fifo_demotion"),
    ("query-key score without the mean over heads", "tests/test_gpu_stream.py", "test_query_key_mode_matches_the_oracle"),
    ("attention received read from the first columns", "tests/test_gpu_stream.py",
     "test_attention_weight_mode_matches_the_oracle"),
]


@pytest.mark.parametrize("what,path,test", CASES, ids=[c[0] for c in CASES])
def test_a_wrong_oracle_fails_the_gpu_parity_test(tmp_path, what, path, test):
    _, old, new = BY_NAME[what]
    src = open(oracle_build.SRC).read()
    assert src.count(old) == 1
    mutant = tmp_path / "ovggt_oracle_mutant.cpp"
    mutant.write_text(src.replace(old, new))
    lib = oracle_build.compile_source(str(mutant), str(tmp_path / "liboracle_mutant.so"))
    env = dict(os.environ, OVGGT_ORACLE_LIBRARY=lib)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, path), "-x", "-q", "-m", "gpu", "-k", test,
                        "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 1, f"the parity test did not notice: {what}\n{r.stdout[-800:]}"
