"""The library built with -DCHICLE_DEBUG_BOUNDS (every index that the solvers and the gap kernels load is checked before
it is used; a failed check ends the call with CHICLE_ERR_INTERNAL) runs the small parity cases: same results, no check
fails. The build under test is chosen when the binding is imported, so the cases run in a process of their own."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CASES = ("test_config1_hinge_dense_full or test_config2_hinge_csr_scaled or test_config3_logistic_dense_scaled or "
         "test_config4_hinge_hashed_elastic_scaled or test_config5_ridge_csc_scaled or test_csr_with_zero_rows or "
         "test_rounds_cut_into_slices or test_lookahead_depths_overlap_modes_and_cluster_sizes or test_dense_shapes or "
         "test_ids_beyond_the_shared_memory_part_across_slices or test_step_budgets_per_partition")


def test_small_parity_cases_under_the_bounds_checking_build():
    from paper_1909_04885_b200 import build
    lib = build.build(debug_bounds=True)
    env = dict(os.environ, CHICLE_LIB_PATH=lib)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"), "-q", "-x", "-m", "gpu",
                        "-k", CASES, "-p", "no:cacheprovider"], env=env, cwd=ROOT, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "deselected" in r.stdout
