"""The debug build of the library (index checks before every gathered load, guard regions between workspace regions)
stands in for a memory checker: the small-corpus parity tests, the Tiny-config tests, the fuzz tests over all three
pipelines, the joint form of stages 1 and 2a and the debug-only checks run once more in a process that loads libchimera_debug.so."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_parity_and_fuzz_tests_pass_under_the_debug_build():
    from paper_2608_23553_b200 import build
    build.build(debug=True)
    env = dict(os.environ, CHIMERA_DEBUG_LIB="1")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_gpu_debug_checks.py"),
           os.path.join(ROOT, "tests", "test_gpu_fuzz.py"),
           os.path.join(ROOT, "tests", "test_gpu_partial.py"),
           os.path.join(ROOT, "tests", "test_gpu_parity.py"),
           os.path.join(ROOT, "tests", "test_gpu_probe_queue.py"),
           "-k", "debug or fuzz or random_configuration or small_corpora or tiny_config_all or parameter_grid or "
                 "stage_isolated or hashed or epilogue or overflowing or joint_stages"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (r.stdout + r.stderr)[-3000:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "skipped" not in r.stdout.splitlines()[-1], tail
