"""The bounds-checking build of the library (-DDELTA_DEBUG_BOUNDS) under a slice of the parity
suite.  In that build every global index the kernels compute by hand is range-checked; an index
out of range is not accessed and DELTA_ERR_BOUNDS lands in the device status word, which the
parity tests read through delta_sparsity_stats.  The slice runs in a child process, because the
binding loads one build of the library per process (DELTA_ATTN_DEBUG_BOUNDS=1 selects this one)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SLICE = ("test_delta_construction_bit_exact or test_device_status_word or "
         "(test_prefill_output_matches_oracle and (T200 or T257 or T700 or T1-)) or "
         "(test_key_delta_decode_steps_match_oracle and (100-64 or 700-128 or 1500-64)) or "
         "(test_decode_steps_match_oracle and (130-64 or 700-64)) or test_bottom_up")


def test_parity_slice_under_the_bounds_checking_build():
    env = dict(os.environ, DELTA_ATTN_DEBUG_BOUNDS="1")
    probe = subprocess.run([sys.executable, "-c",
                            "from paper_2507_19608_b200 import binding as B; print(B.lib.delta_debug_bounds_build())"],
                           cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert probe.returncode == 0 and probe.stdout.strip() == "1", probe.stderr[-2000:]
    r = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "-m", "gpu", "-x", "-q", "-k", SLICE],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1800)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-1000:]
    assert " passed" in r.stdout
