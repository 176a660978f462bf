"""The checked build of the library (-DPLORA_DEBUG): every address a kernel forms from a table, a work unit or a
token index is compared with its buffer before use, and a violation would show as PLORA_ERR_DEBUG_CHECK in the
status word.  It stands in for a memory checker, which cannot be run on the test machines.  The library is chosen
when it is loaded, so the shape-heavy parity cases run again in a child process with PLORA_DEBUG_BUILD=1; they assert
a zero status word themselves."""
import os
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu

ROOT = Path(__file__).resolve().parent.parent
CASES = ("tiny_config or odd_ranks or ragged_dims or token_counts or sgmv_tile_shapes or random_shapes or "
         "mixed_rank_calls or grouped_projections or three_long_segments or empty_and_all_minus_one or "
         "shrink_and_expand_entry_points or two_byte_m or out_of_range_id or inputs_resident_hint or both_kinds")


def test_parity_cases_pass_under_the_checked_build():
    env = dict(os.environ, PLORA_DEBUG_BUILD="1")
    which = subprocess.run([sys.executable, "-c", "import paper_2608_05483_b200 as P; P.load(); print(P.library_path().name)"],
                           cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert which.returncode == 0, which.stderr[-2000:]
    assert which.stdout.strip().endswith("libplora_b200_debug.so")
    run = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "-x", "-q", "-m", "gpu", "-k", CASES,
                          "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert run.returncode == 0, run.stdout[-3000:] + run.stderr[-1000:]
    assert " passed" in run.stdout and "failed" not in run.stdout
