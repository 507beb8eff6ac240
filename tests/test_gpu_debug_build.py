"""The bounds-checked build of the library (env kernel compiled -DIM_DEBUG: every index it forms from its inputs is
tested and reported in the status word instead of being dereferenced).  It stands in for a memory checker: the
small parity cases -- ragged batches, tiny and wide skeletons, every optional semantic, resets with write-back --
run against it in a process of their own, and each of their steps asserts a clean status word."""
import os
import subprocess
import sys

import pytest

from paper_2609_09821_b200 import build as lib_build

pytestmark = pytest.mark.gpu

CASES = [
    "tests/test_gpu_parity.py::test_cfg1_tiny_fp32_full",
    "tests/test_gpu_parity.py::test_ragged_batches",
    "tests/test_gpu_parity.py::test_single_body_and_max_bodies",
    "tests/test_gpu_parity.py::test_min_ld_obs_and_padded_component_stride",
    "tests/test_gpu_parity.py::test_all_reset_and_none_reset",
    "tests/test_gpu_edge_cases.py::test_all_optional_semantics_together",
    "tests/test_gpu_edge_cases.py::test_skeletons_with_more_than_eight_leaves",
    "tests/test_gpu_edge_cases.py::test_two_keyframe_clips_reset_every_step",
    "tests/test_gpu_edge_cases.py::test_training_summaries_accumulate_on_the_device",
]


def test_small_parity_cases_are_clean_under_the_bounds_checked_build():
    path = lib_build.build(debug=True) and lib_build.DEBUG_LIB_PATH
    assert os.path.exists(path)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, IM_B200_LIB=path)
    out = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider"] + CASES, cwd=root, env=env,
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-2000:]
    assert " passed" in out.stdout
