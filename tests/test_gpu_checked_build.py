"""The range-checked build of the library (-DDRK_BOUNDS_CHECK) on a GPU.

compute-sanitizer is not available on the machines these tests run on, so the library carries its own checks: in
the checked build every index that a kernel derives from device-side data (row maps, compacted row counts,
work-unit numbers, store coordinates) is compared with its array's extent before use; a violation sets
DRK_STATUS_BOUNDS and skips the access.  Here a subset of the parity and edge tests runs against that build in
a child process (the library is chosen per process); they assert a zero status word, hence no violation, on
sizes ragged in every dimension, compacted backward rows, vocabulary ranges and the forward over usable rows."""
import os
import subprocess
import sys

import pytest

from paper_2602_05885_b200 import build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SUBSET = [
    "tests/test_gpu_edge.py::test_ragged_sizes",
    "tests/test_gpu_edge.py::test_all_rejected_gives_exact_zero",
    "tests/test_gpu_edge.py::test_empty_inputs",
    "tests/test_gpu_parity.py::test_bf16_shapes[0-medium]",
    "tests/test_gpu_parity.py::test_bf16_shapes[2-medium]",
    "tests/test_gpu_parity.py::test_forward_over_usable_rows_only",
    "tests/test_gpu_shards.py::test_bf16_in_ranges",
    "tests/test_gpu_trloo.py",
]


def test_parity_subset_on_the_checked_build():
    lib = build.build_library(bounds_check=True)
    env = dict(os.environ, DRK_LIBRARY=lib)
    probe = subprocess.run([sys.executable, "-c", "from paper_2602_05885_b200 import binding as B; "
                            "print(B.drk_bounds_checked(), B.library_path())"], cwd=ROOT, env=env,
                           capture_output=True, text=True, timeout=300)
    assert probe.returncode == 0 and probe.stdout.split()[0] == "1", probe.stdout + probe.stderr
    res = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider"] + SUBSET,
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
