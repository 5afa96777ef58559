"""The small-case subset of the GPU parity tests under the library built with index checks.

No memory checker can be run on the kernels, so the library has a debug build
(`python -m paper_2211_04515_b200.build --check`, -DQP_CHECK_BOUNDS) in which every index into the
kernels' shared-memory tables and scratch rows is range-checked: an index out of range is redirected
to entry 0 (nothing traps, nothing faults) and raises QP_DEV_INDEX_RANGE in what qp_get_status
returns.  This test builds that variant, runs the small cases (c1, ragged sizes, degenerate and
non-finite inputs, searches at 1 to 8 bits, channel-wise and token-wise shapes) in a child process
that loads it through QUANTPIPE_LIB, and expects them to pass with the bit clear (the child's
conftest checks the bit once more at the end of the session).
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu

SUBSET = ("test_stats_configs or test_stats_ragged or test_stats_special or stats_one_launch or test_pack_unpack_c1 or "
          "test_pack_unpack_ragged or test_pack_special or test_search_c1 or test_search_steps or "
          "test_search_ragged or test_search_degenerate or test_fused_sender_c1 or fused_sender_special or "
          "test_channels_shapes or test_search_channels_vit or test_tokens_shapes")


def test_small_cases_run_clean_under_the_index_checked_build():
    from paper_2211_04515_b200 import build
    lib = build.build(check=True)
    env = dict(os.environ, QUANTPIPE_LIB=lib)
    run = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "-m", "gpu", "-q", "-x", "-k", SUBSET],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (run.stdout or "")[-3000:] + (run.stderr or "")[-2000:]
    assert run.returncode == 0, tail
    assert " passed" in run.stdout and "index checks: on, no index out of range" in run.stdout, tail
