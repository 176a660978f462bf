"""The parity cases once more with the inputs-resident hint switched on in every context the tests build
(gpu_util.Runner reads PLORA_TEST_INPUTS_RESIDENT): the fused launches then use the kernels that read x and
start multiplying before they join the stream order.  The cases assert parity with the oracle, bit-for-bit
repeatability and a zero status word themselves; here they run in a child process with the variable set."""
import os
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu

ROOT = Path(__file__).resolve().parent.parent
CASES = ("tiny_config or reduced_benchmark_configs or odd_ranks or ragged_dims or token_counts or random_shapes or "
         "mixed_rank_calls or cuda_graph_replay or grouped_projections or half_precision or auto_dispatch or "
         "three_long_segments or empty_and_all_minus_one or out_of_range_id or both_kinds")


def test_parity_cases_pass_with_the_hint_on():
    env = dict(os.environ, PLORA_TEST_INPUTS_RESIDENT="1")
    run = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "-x", "-q", "-m", "gpu", "-k", CASES,
                          "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert run.returncode == 0, run.stdout[-3000:] + run.stderr[-1000:]
    assert " passed" in run.stdout and "failed" not in run.stdout
