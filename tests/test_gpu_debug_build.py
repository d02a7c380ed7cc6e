"""The bounds-checked flavour of the library (-DNB_DEBUG, libnb_debug.so) under a slice of the GPU suite.

Every kernel of that flavour range-checks each tile coordinate, ring slot, table index and global
address before it uses it; a failed check records a code that nb_check_guards (called at the end of
the parity tests) reports.  The tests run in a child process because the binding picks its library
once, at import, from NB_LIB_PATH."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_a_slice_of_the_gpu_suite_passes_under_the_bounds_checked_library():
    from paper_2211_00889_b200.build import build_library
    lib = build_library(flavour="debug")
    env = dict(os.environ, NB_LIB_PATH=lib)
    probe = subprocess.run([sys.executable, "-c",
                            "from paper_2211_00889_b200 import binding as B; print(B.lib.nb_debug_build())"],
                           cwd=ROOT, env=env, capture_output=True, text=True)
    assert probe.returncode == 0 and probe.stdout.strip() == "1", probe.stderr[-2000:]
    picked = ("sizes_around_one_tile or unaligned_rows_against_the_oracle or short_range_kernel or "
              "aligned_and_unaligned_streams or more_minibatches or learner_counts or matcha_and_options or "
              "streaming_hold or cfg1_tiny or centralized_step_on_pipeline_sizes")
    run = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-k", picked,
                          "tests/test_gpu_pipeline.py", "tests/test_gpu_parity.py"],
                         cwd=ROOT, env=env, capture_output=True, text=True)
    assert run.returncode == 0, run.stdout[-3000:] + run.stderr[-2000:]
    assert " passed" in run.stdout and "failed" not in run.stdout
