"""The index-checking build (-DCLADA_DEBUG_BOUNDS): every neuron index is range-checked on its way into a row
address or a list slot, a bad one raises CLADA_STATUS_BAD_INDEX in the call's status word and is made harmless.
Parity cases of the decode calls (one sequence, the stack launch, tiles, nested lists, and the dense pass, which
gathers nothing) run on that build in a child process: they pass against the oracle as on the release build, and the status words they
assert on stay 0 -- no check fires on any list the kernels build themselves.
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CASES = [
    "tests/test_gpu_parity.py::test_sparse_ffn_bf16_shapes",
    "tests/test_gpu_parity.py::test_sparse_ffn_f32_shapes",
    "tests/test_gpu_parity.py::test_sparse_ffn_degenerate_thresholds_and_determinism",
    "tests/test_gpu_parity.py::test_sparse_ffn_batched_tiles",
    "tests/test_gpu_parity.py::test_algorithm2_loop_config1",
    "tests/test_gpu_batch_dense.py::test_dense_pass_matches_oracle",
    "tests/test_gpu_batch_dense.py::test_stack_call_with_a_batch_runs_dense_passes",
    "tests/test_gpu_stack.py",
    "tests/test_gpu_nested.py",
]


def test_parity_cases_pass_on_the_index_checking_build():
    from paper_2502_19078_b200 import build
    lib = build.build(variant="bounds")
    env = dict(os.environ, CLADA_LIB=lib)
    done = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider"] + CASES,
                          cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    tail = done.stdout[-3000:] + done.stderr[-1000:]
    assert done.returncode == 0, tail
    assert " passed" in done.stdout and "failed" not in done.stdout, tail
