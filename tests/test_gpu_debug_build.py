"""The checked build of the library (every computed index range-checked, histogram and candidate counts
checked for conservation; a failed check sets the status word, nothing traps) under the tiny, adversarial and
clustered parity cases.  The cases run in a child pytest process whose binding loads libiwp_debug.so; each of
them already asserts a clean status word and bit-exact parity with the oracle."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_parity_cases_on_the_checked_build():
    sys.path.insert(0, ROOT)
    from paper_1901_01544_b200 import build as lib_build

    lib_build.build(debug=True)
    env = dict(os.environ, IWP_LIB_VARIANT="debug", IWP_SHAPE_SEEDS="4", IWP_WALK_SEEDS="1")
    which = subprocess.run([sys.executable, "-c", "from paper_1901_01544_b200 import binding; print(binding.LIB_PATH)"],
                           cwd=ROOT, env=env, capture_output=True, text=True)
    assert which.returncode == 0 and which.stdout.strip().endswith("libiwp_debug.so"), which.stdout + which.stderr
    cases = ("test_random_values or test_many_ties or test_degenerate_layers or test_forced_scalar or test_exact_select "
             "or test_misaligned or test_random_shapes or test_zero_weight_block or test_run_lengths or "
             "test_hot_gradient_run or test_many_dense or test_union_of_several or test_leader_only_select")
    r = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "tests/test_gpu_clustered.py", "-q", "-x",
                        "-m", "gpu", "-k", cases, "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True)
    assert r.returncode == 0, r.stdout[-4000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and " failed" not in r.stdout
