"""The -DDAD_BOUNDS_CHECK build of the library as its own memory checker (compute-sanitizer cannot be run where
these tests run): every global access of the kernels that compute their own indices is tested against the address
ranges the entry points registered.  In-bounds code must leave the record empty and the results unchanged; with
every range cut short by 64 bytes (DAD_BOUNDS_SHRINK) the accesses to those last bytes -- legitimate ones -- must be
caught, skipped and recorded, without a trap or a fault."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


def run_driver(extra_env):
    sys.path.insert(0, ROOT)
    from paper_2102_09631_b200 import build
    build.build_check()
    env = dict(os.environ, DAD_LIB="libdad_check.so", **extra_env)
    res = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "bounds_check_driver.py")], env=env,
                         capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    return json.loads(res.stdout.strip().splitlines()[-1])


def test_in_bounds_code_leaves_no_record_and_the_results_stand():
    out = run_driver({})
    assert out["violations"] == 0, out
    assert out["worst_error_over_bar"] <= 1.0


def test_shortened_ranges_are_caught_without_a_fault():
    out = run_driver({"DAD_BOUNDS_SHRINK": "64"})
    assert out["violations"] > 0 and out["first_bytes"] in (2, 4, 8, 16) and out["first_line"] > 0
