"""Are the oracle's pins tight?  One mistake at a time is planted in a COPY of the oracle's source (on the CPU, in a
temporary folder), the copy is compiled, and the pins of tests/test_oracle_pins.py are run against it in a child
process: every planted mistake has to make some pin fail.  Each entry gives the exact source text it replaces, so
an entry that no longer matches the source fails loudly instead of turning into a mutant that changes nothing."""
import os
import subprocess
import sys

import pytest

from oracle import build as oracle_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

MISTAKES = [
    ("Eq. 5 without the square root", "s[j] = std::sqrt(acc);", "s[j] = acc;"),
    ("Eq. 6 with alpha and 1 - alpha swapped", "alpha * conv + (1.0 - alpha) * raw", "(1.0 - alpha) * conv + alpha * raw"),
    ("Eq. 6 with rows and columns of the map swapped", "S[(size_t)yy * grid_w + xx]", "S[(size_t)xx * grid_h + yy]"),
    ("diversity as the cosine itself", "d[i] = 1.0 - cosine(ki, kbar.data(), C);", "d[i] = cosine(ki, kbar.data(), C);"),
    ("Eq. 7 with the two weights swapped",
     "minmax_group(d, flags, n, 1.0 - beta, r);\n  minmax_group(s, flags + n, M, beta, r + n);",
     "minmax_group(d, flags, n, beta, r);\n  minmax_group(s, flags + n, M, 1.0 - beta, r + n);"),
    ("Eq. 7 with protected rows inside the min-max range",
     "if (flags[i] == ORC_FLAG_EVICTABLE) {\n      lo = std::min(lo, x[i]);", "if (true) {\n      lo = std::min(lo, x[i]);"),
    ("Eq. 8 with ties going to the higher position",
     "return rank_key(r[a]) > rank_key(r[b]); });\n  std::vector<int32_t> keep(prot);",
     "return rank_key(r[a]) > rank_key(r[b]) || (rank_key(r[a]) == rank_key(r[b]) && a > b); });\n"
     "  std::vector<int32_t> keep(prot);"),
    ("Eq. 8 with a budget that forgets the protected rows",
     "int64_t k = (int64_t)B - (int64_t)prot.size();", "int64_t k = (int64_t)B;"),
    ("attention without 1 / sqrt(d)",
     "const double scale = 1.0 / std::sqrt((double)head_dim);\n  const int64_t work", "const double scale = 1.0;\n  const int64_t work"),
    ("attention reading V of the neighbouring head",
     "(double)V[(size_t)n * C + (size_t)h * head_dim + c]", "(double)V[(size_t)n * C + (size_t)((h + 1) % n_heads) * head_dim + c]"),
    ("FIFO that drops the newest anchor",
     "demoted = st->anchors.front();\n      st->anchors.pop_front();", "demoted = st->anchors.back();\n      st->anchors.pop_back();"),
    ("anchor interval off by one", "t - st->last_registration >= cfg.min_anchor_interval", "t - st->last_registration > cfg.min_anchor_interval"),
    ("anchor tokens flagged without the offset of the special tokens",
     "st->flags[n + cfg.n_special + p] = ORC_FLAG_HIST;", "st->flags[n + p] = ORC_FLAG_HIST;"),
    ("stored score taken before smoothing", "st->stored[n + j] = (float)s_smooth[j];", "st->stored[n + j] = (float)s[j];"),
    ("random priority that ignores the token", "orc_splitmix64(step_key + (uint64_t)token_id)", "orc_splitmix64(step_key)"),
    ("query-key score without the mean over heads", "s[j] = total / ((double)M * (double)n_heads);", "s[j] = total / ((double)M);"),
    ("attention received read from the first columns", "s[j] += p[first_col + j] / denom;", "s[j] += p[j] / denom;"),
]


@pytest.mark.parametrize("what,old,new", MISTAKES, ids=[m[0] for m in MISTAKES])
def test_a_planted_mistake_fails_a_pin(tmp_path, what, old, new):
    src = open(oracle_build.SRC).read()
    assert src.count(old) == 1, f"the source text this entry replaces has changed: {what}"
    mutant = tmp_path / "ovggt_oracle_mutant.cpp"
    mutant.write_text(src.replace(old, new))
    lib = oracle_build.compile_source(str(mutant), str(tmp_path / "liboracle_mutant.so"))
    env = dict(os.environ, OVGGT_ORACLE_LIBRARY=lib)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"), "-x", "-q",
                        "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 1, f"no pin noticed: {what}\n{r.stdout[-600:]}"
