"""The checked build of the library (-DCONCUR_BOUNDS) stands in for a memory checker: its kernels hold
every index they compute for the workspace, the partial buffers and the outputs against the buffer's
capacity and record a violation instead of making the access.  Here the edge-length, cascade, layer and
KV-head parity cases are run once more in a child process that loads that build; each of them asserts
that the device flags are zero, so a single out-of-range index anywhere fails the run."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu

CASES = [
    "tests/test_gpu_parity.py::test_edge_lengths_and_forced_splits",
    "tests/test_gpu_parity.py::test_many_short_sequences",
    "tests/test_gpu_parity.py::test_batch_sizes_around_the_in_kernel_plan_limits",
    "tests/test_gpu_cascade.py::test_cascade_matches_oracle",
    "tests/test_gpu_cascade.py::test_long_shared_prefix_split_over_many_ctas",
    "tests/test_gpu_cascade.py::test_malformed_group_tables_share_nothing_and_are_flagged",
    "tests/test_gpu_prefill.py",
    "tests/test_gpu_layers.py",
    "tests/test_gpu_kv_heads.py::test_plain_step",
    "tests/test_kv_append.py",
]


def test_parity_cases_pass_on_the_checked_build_with_no_index_out_of_bounds():
    sys.path.insert(0, ROOT)
    from paper_2510_07356_b200 import build
    lib = build.build_bounds()
    env = dict(os.environ, CONCUR_ATTN_LIBRARY=str(lib))
    pr = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider", *CASES],
                        cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert pr.returncode == 0, pr.stdout[-3000:] + pr.stderr[-1000:]
    assert " passed" in pr.stdout


def test_the_checked_build_is_what_the_child_loads():
    sys.path.insert(0, ROOT)
    from paper_2510_07356_b200 import build
    lib = build.build_bounds()
    code = ("import paper_2510_07356_b200.binding as b, os; "
            "assert str(b._LIB_PATH) == os.environ['CONCUR_ATTN_LIBRARY'], b._LIB_PATH; print('ok')")
    pr = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=dict(os.environ, CONCUR_ATTN_LIBRARY=str(lib)),
                        capture_output=True, text=True, timeout=300)
    assert pr.returncode == 0 and "ok" in pr.stdout, pr.stderr[-1000:]
