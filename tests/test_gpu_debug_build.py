"""The small parity cases once more under the library built with -DPQHSA_DEBUG (-m gpu).

That build records, in the status word, every index that the release build silently clamps or
skips (list id >= n_list, selected position outside the indexed region, negative page id).  On
valid inputs the word must stay 0 and the results must not change.  The checks never trap, and
no test feeds the GPU a bad index on purpose: the predicates themselves are unit-tested on the
host (test_abi_host.py)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CASES = ("c1 or ragged_batch_with_empty or sinks_window_pages_ragged or paper_index_4bit or "
         "g16_four_head_groups or pages_of_1 or lists_4096_mostly_empty or norm_jump")


def test_small_cases_under_the_debug_build_leave_the_status_word_clear():
    from paper_2609_33746_b200.build import build_library
    lib = build_library(debug=True)                  # built by __graft_entry__.build(); rebuilt if stale
    env = dict(os.environ, PQHSA_LIBRARY=lib)
    probe = subprocess.run(
        [sys.executable, "-c",
         "from paper_2609_33746_b200 import pqhsa; import sys; sys.exit(0 if pqhsa.debug_build() else 3)"],
        cwd=ROOT, env=env)
    assert probe.returncode == 0, "PQHSA_LIBRARY did not select the debug build"
    # test_stage_attend_and_fused_decode and test_stage_select assert device_status() == OK
    r = subprocess.run(
        [sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "-x", "-q", "-m", "gpu", "-k",
         f"(stage_attend or stage_select) and ({CASES})"],
        cwd=ROOT, env=env, capture_output=True, text=True)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
