"""The pins must fail when the oracle is wrong.

Each case plants one plausible mistake in a copy of ``oracle/mor_oracle.c`` (a dropped rule, a wrong
comparison, a wrong constant), builds it in a temporary directory and runs the pin files against that
copy in a child process.  The case passes when the pins FAIL.  Nothing here touches the real oracle
library or the GPU.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "mor_oracle.c")

# (name, text in the source, replacement, pin files that must catch it)
MISTAKES = [
    ("eq3_tie_rejects_e4m3", "(b->sum_rel_e4m3 <= b->sum_rel_e5m2)", "(b->sum_rel_e4m3 < b->sum_rel_e5m2)",
     ["tests/test_oracle_mor.py"]),
    ("alg1_exponent_lowered_on_equal_mantissas", "if (!(m_g <= m_b)) e -= 1;", "if (!(m_g < m_b)) e -= 1;",
     ["tests/test_oracle_gam.py"]),
    ("eq4_bound_without_the_subnormals", "b->amax < 939524096.0 * mn", "b->amax < 234881024.0 * mn",
     ["tests/test_oracle_mor.py"]),
    ("zeros_counted_in_the_sums", "if (bf16_is_zero(h)) continue;          /* sums of Eq. 1-3 run over x != 0 */", "",
     ["tests/test_oracle_mor.py"]),
    ("eq2_not_strict_for_a_block", "return err < cfg->threshold ? ORC_FMT_E4M3 : ORC_FMT_BF16;",
     "return err <= cfg->threshold ? ORC_FMT_E4M3 : ORC_FMT_BF16;", ["tests/test_oracle_mor.py"]),
    ("eq2_not_strict_for_the_tensor", "t.mean_rel_e4m3 < cfg->threshold", "t.mean_rel_e4m3 <= cfg->threshold",
     ["tests/test_oracle_mor.py"]),
    ("bf16_rounding_half_up", "u += 0x7FFFu + ((u >> 16) & 1u);", "u += 0x8000u;",
     ["tests/test_oracle_fake_quant.py"]),
    ("e5m2_scale_six_binades_up", "uint32_t e5 = e + 7 > 254 ? 254 : e + 7;", "uint32_t e5 = e + 6 > 254 ? 254 : e + 6;",
     ["tests/test_oracle_mor.py", "tests/test_oracle_gam.py"]),
]


def run_pins(tmp_path, source_text, files):
    src = tmp_path / "mor_oracle.c"
    src.write_text(source_text)
    env = dict(os.environ, MOR_ORACLE_SRC=str(src), MOR_ORACLE_LIB=str(tmp_path / "libmor_oracle.so"))
    return subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", *files],
                          cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)


def test_the_unchanged_copy_passes(tmp_path):
    """The child-process arrangement itself: an unchanged copy of the source is green."""
    r = run_pins(tmp_path, open(SRC).read(), ["tests/test_oracle_gam.py", "tests/test_oracle_fake_quant.py"])
    assert r.returncode == 0, r.stdout[-2000:]


@pytest.mark.parametrize("name,old,new,files", MISTAKES, ids=[m[0] for m in MISTAKES])
def test_a_planted_mistake_is_caught(tmp_path, name, old, new, files):
    text = open(SRC).read()
    assert text.count(old) == 1, f"{name}: the line to change is not in the source (or not unique)"
    r = run_pins(tmp_path, text.replace(old, new), files)
    assert r.returncode == 1, f"{name}: the pins did not fail\n" + r.stdout[-1500:]
    assert " failed" in r.stdout
