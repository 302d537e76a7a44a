"""The candidate-checking tool accepts the library itself and reports a disagreement with the oracle."""
import json
import os
import subprocess
import sys

import pytest

from paper_2509_07506_b200 import build as astra_build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TOOL = os.path.join(ROOT, "tests", "check_candidate.py")


def run(lib, *extra):
    out = subprocess.run([sys.executable, TOOL, "--lib", lib, *extra], capture_output=True, text=True, timeout=900)
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert lines, out.stderr[-2000:]
    return out.returncode, json.loads(lines[-1])


def test_library_passes_its_own_check():
    rc, rec = run(astra_build.build(), "--round", "1", "--baseline", astra_build.build())
    # worst_ulp is relative to |oracle|, which can be tiny where the merge blend cancels (the gate adds a floor there)
    assert rc == 0 and rec["correct"] and rec["cases"] == 34 and rec["worst_ulp"] > 0
    assert len(rec["performance"]["us_per_call"]) == 12 and rec["performance"]["geomean_us"] > 0
    assert 0.5 < rec["geomean_speedup_over_baseline"] < 2.0


def test_disagreement_with_the_oracle_is_reported(tmp_path):
    """Validation must fail when candidate and oracle disagree.  The disagreement is planted in a copy
    of the ORACLE (its epsilon dropped), on the CPU; the candidate is the unmodified library."""
    import oracle
    src = open(os.path.join(os.path.dirname(os.path.abspath(oracle.__file__)), "astra_oracle.c")).read()
    bad = src.replace("sqrt(sum_sq / (double)H + (double)eps)", "sqrt(sum_sq / (double)H + 0.5)")
    assert bad != src
    bad_src = tmp_path / "oracle_bad.c"
    bad_src.write_text(bad)
    bad_lib = oracle.compile_source(str(bad_src), str(tmp_path / "liboracle_bad.so"))
    rc, rec = run(astra_build.build(), "--oracle-lib", bad_lib)
    assert rc == 1 and not rec["correct"] and any("rmsnorm" in f for f in rec["failures"])
