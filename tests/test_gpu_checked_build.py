"""The bounds-checked build of the library (libspsyrk_checked.so: every shared-memory slot and output
offset the kernels compute is tested before it is used; a violation is reported as an internal
error instead of touching memory) must run the reduced workloads, the mirror and the random-matrix
sweep clean: every call returns SPSYRK_OK and every result still matches the oracle.  The selected
tests are run once more in a child process that loads that build."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CHECKED = os.path.join(ROOT, "paper_2608_09713_b200", "libspsyrk_checked.so")


def test_checked_build_runs_clean():
    from paper_2608_09713_b200 import build
    assert build.build_cuda(checked=True) == CHECKED      # rebuilt here when a source is newer than the library
    env = dict(os.environ, SPSYRK_LIBRARY=CHECKED)
    probe = subprocess.run([sys.executable, "-c", "from paper_2608_09713_b200 import binding as B; print(B.LIB_PATH)"],
                           cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert probe.returncode == 0 and probe.stdout.strip() == CHECKED, probe.stderr[-2000:]
    sel = ["tests/test_gpu_parity.py::test_small_configs", "tests/test_gpu_parity.py::test_mirror",
           "tests/test_gpu_parity.py::test_rows_at_every_class_boundary", "tests/test_gpu_parity.py::test_blocks",
           "tests/test_gpu_parity.py::test_symm", "tests/test_gpu_parity.py::test_one_pass_mode",
           "tests/test_gpu_parity.py::test_numeric_by_row_blocks", "tests/test_gpu_parity.py::test_mirror_general_lower_triangles",
           "tests/test_gpu_random.py"]
    run = subprocess.run([sys.executable, "-m", "pytest", *sel, "-m", "gpu", "-x", "-q", "-p", "no:cacheprovider"],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=3000)
    assert run.returncode == 0, run.stdout[-4000:] + run.stderr[-2000:]
    assert " passed" in run.stdout and "failed" not in run.stdout
