"""The tensor-core GEMMs can run as cluster pairs (two CTAs per MMA, TRL_CTA_GROUP=2).  The setting
is read once per process, so the parity tests are run again in a child process with it on."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_parity_tests_pass_with_cta_pairs():
    env = dict(os.environ, TRL_CTA_GROUP="2")
    probe = subprocess.run([sys.executable, "-c", "import paper_2510_17891_b200 as t; print(t.trl_config_string())"],
                           cwd=ROOT, env=env, capture_output=True, text=True)
    assert probe.returncode == 0 and "cta_group_fwd=2 cta_group_bwd=2" in probe.stdout, probe.stdout + probe.stderr
    sel = ("ragged_multi_tile or many_tiles or long_reasoning_twin or fused_step_matches_oracle or edge_cases or "
           "smallest_legal or minimum_workspace or degenerate or all_equal or confident_policy_every or inactive_row_blocks")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "tests/test_gpu_parity_small.py", "-k", sel],
                       cwd=ROOT, env=env, capture_output=True, text=True)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "no tests ran" not in r.stdout
