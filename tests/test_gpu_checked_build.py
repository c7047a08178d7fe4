"""The parity tests once more on the checked build of the library (-DPODS_BOUNDS_CHECK): every index a kernel computes
is compared with its extent, and a violation raises PODS_STATUS_INTERNAL instead of touching memory.  This stands in
for a memory checker: the tests below assert a clean status word on clean inputs, so a stray index fails them even
when it would have landed on harmless memory in the normal build."""
import os
import subprocess
import sys

import pytest

from paper_2504_13818_b200.csrc import build as cuda_build

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SUBSET = ["tests/test_gpu_select.py", "tests/test_gpu_compact.py", "tests/test_gpu_accumulation.py",
          "tests/test_gpu_lm_head.py::test_logp_against_the_oracle_on_all_rows",
          "tests/test_gpu_lm_head_loss.py::test_loss_and_gradients_against_the_oracle",
          "tests/test_gpu_lm_head_loss.py::test_several_panels_accumulate_to_the_same_result",
          "tests/test_gpu_loss.py::test_config1_whole_path_values",
          "tests/test_gpu_loss.py::test_vocab_sizes_span_tiles_and_ragged_tails",
          "tests/test_gpu_loss.py::test_cluster_path_vocab_sizes",
          "tests/test_gpu_loss.py::test_masked_rows_and_empty_rollouts"]


def test_parity_subset_on_the_checked_build():
    lib = cuda_build.CHECKED_LIB
    sources = cuda_build.SOURCES + cuda_build.HEADERS
    if not os.path.exists(lib) or any(os.path.getmtime(f) > os.path.getmtime(lib) for f in sources):
        cuda_build.build(checked=True)
    env = dict(os.environ, PODS_B200_LIBRARY=lib)
    out = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider"] + SUBSET,
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-1000:]
    assert " passed" in out.stdout


def test_the_checked_build_is_the_one_that_was_loaded():
    """The override is honoured: a process started with PODS_B200_LIBRARY reports that path."""
    lib = cuda_build.CHECKED_LIB
    if not os.path.exists(lib):
        cuda_build.build(checked=True)
    code = "from paper_2504_13818_b200 import binding; binding.load(); print(binding.LIB_PATH)"
    out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=dict(os.environ, PODS_B200_LIBRARY=lib),
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip().endswith("libpods_b200_checked.so"), out.stdout + out.stderr
