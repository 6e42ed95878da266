"""The bounds-checked build of the library (every computed position checked, violations reported through
UNCOMP_STATUS_BOUNDS and skipped) must run the small parity cases with a clean status word and the same results.

The library is chosen when the binding is imported, so the cases run in a child process with
UNCOMP_DEBUG_LIBRARY=1; the child is the ordinary parity suite restricted to its small cases."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_parity_cases_on_the_debug_library():
    from paper_2410_03090_b200 import build
    build.build(debug=True)
    env = dict(os.environ, UNCOMP_DEBUG_LIBRARY="1")
    cases = ["tests/test_gpu_parity.py::test_config1_fp32_whole_pass",
             "tests/test_gpu_parity.py::test_bf16_small_whole_pass",
             "tests/test_gpu_parity.py::test_select_extreme_budgets",
             "tests/test_gpu_parity.py::test_select_ties_take_lowest_positions",
             "tests/test_gpu_evict.py", "tests/test_gpu_decode.py"]
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider"] + cases,
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    # the child really ran on the debug library
    probe = subprocess.run([sys.executable, "-c",
                            "from paper_2410_03090_b200 import binding; print(binding.lib._name)"],
                           cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert "libuncomp_debug.so" in probe.stdout, probe.stdout + probe.stderr
