"""The library's alternative forms are selected by environment variables that are read once per
process (tuning aids: the unpaired tensor-core kernel, stream launches instead of graph replay for the
refresh, no small-order lanes).  Each is exercised here in a child process that runs a few of the
ordinary parity tests under that setting, so that the forms a user can fall back to stay correct."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(env, args):
    e = dict(os.environ)
    e.update(env)
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider"] + args,
                       cwd=ROOT, env=e, capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]


def test_unpaired_tensor_core_kernel():
    _run({"BR_TC_PAIR": "0"}, ["tests/test_gpu_gemm_tc.py",
                               "tests/test_gpu_full_size.py::test_c2_full_size_block_teacher_forced_bases"])


def test_refresh_without_graphs_and_small_lanes():
    _run({"BR_REFRESH_GRAPHS": "0", "BR_REFRESH_SMALL_LANES": "0", "BR_REFRESH_LANES": "1"},
         ["tests/test_gpu_full_size.py::test_refresh_order_1024_against_oracle_power",
          "tests/test_gpu_full_size.py::test_refresh_tensor_core_projections",
          "tests/test_gpu_parity_fp32.py::test_numerically_rank_deficient_refresh_is_completed_in_the_same_call",
          "tests/test_gpu_parity_bf16.py", "-k", "not checkpoint"])
