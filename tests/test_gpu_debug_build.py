"""The bounds-checked debug build (libtrl_debug.so, -DTRL_DEBUG_BOUNDS) checks every store whose index
comes out of the row packing against its buffer and flags TRL_ERR_BOUNDS instead of storing.  The
parity tests read the status word after every call, so running them against that build shows that no
such store ever leaves its buffer, on ragged, chunked, banded and inactive-block cases alike.  The
build is chosen per process (TRL_DEBUG_BUILD=1), hence the child process."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_parity_tests_pass_on_the_bounds_checked_build_without_a_violation():
    from paper_2510_17891_b200 import build
    assert os.path.exists(build.build(debug=True))
    env = dict(os.environ, TRL_DEBUG_BUILD="1")
    probe = subprocess.run([sys.executable, "-c",
                            "import paper_2510_17891_b200 as t; t.load_library(); print(t.binding.lib_path()); "
                            "print(t.trl_status_string(11))"], cwd=ROOT, env=env, capture_output=True, text=True)
    assert probe.returncode == 0 and "libtrl_debug.so" in probe.stdout and "debug build" in probe.stdout, probe.stdout + probe.stderr
    sel = ("ragged_multi_tile or many_tiles or long_reasoning_twin or fused_step_matches_oracle or edge_cases or "
           "smallest_legal or minimum_workspace or degenerate or inactive_row_blocks or config0 or many_rollouts")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "tests/test_gpu_parity_small.py",
                        "tests/test_gpu_banded.py", "-k", sel + " or banded"],
                       cwd=ROOT, env=env, capture_output=True, text=True)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "no tests ran" not in r.stdout
