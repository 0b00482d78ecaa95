"""The bounds-checking build (-DXG_DEBUG_BOUNDS): config C1 along its whole trajectory, the exhaustive small-grammar
suite and the capacity cases run on it in a child process; every mask still equals the oracle's and no range check
of any kernel fails (tests/conftest.py asks the library after every test)."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu


def test_parity_suites_pass_on_the_bounds_checking_library():
    env = dict(os.environ, XG_DEBUG_BOUNDS="1")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu",
           os.path.join(ROOT, "tests", "test_gpu_small_grammars.py"),
           os.path.join(ROOT, "tests", "test_gpu_parity.py") + "::test_c1_every_step_bit_exact",
           os.path.join(ROOT, "tests", "test_gpu_parity.py") + "::test_c5_recursive_json_with_utf8",
           os.path.join(ROOT, "tests", "test_gpu_parity.py") + "::test_item_sets_beyond_the_fast_path",
           os.path.join(ROOT, "tests", "test_gpu_parity.py") + "::test_long_tokens_up_to_255_bytes",
           os.path.join(ROOT, "tests", "test_gpu_fused_step.py") + "::test_fill_and_apply_with_a_ragged_vocabulary"]
    out = subprocess.run(cmd, capture_output=True, text=True, env=env, cwd=ROOT, timeout=1500)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-2000:]
    assert " passed" in out.stdout


def test_the_regular_library_has_no_checks():
    from paper_2601_04426_b200 import binding as B
    if os.environ.get("XG_DEBUG_BOUNDS") == "1":
        pytest.skip("this process runs on the checking build")
    assert B.lib().xg_debug_bounds_enabled() == 0
    B.debug_bounds_check()
