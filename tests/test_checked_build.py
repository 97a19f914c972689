"""The checked build of the library (-DASYNCLM_DEBUG): every page id a kernel turns into an address is
compared with the pool's size on the device; a bad one sets the plan's status word and the access is
left out, so nothing faults.  The planner already rejects bad ids on the host, so the test overwrites
one id in the plan's device copy after planning, in a child process that has loaded the checked build
only (the ordinary build has no such check and must never see that plan)."""
import json
import os
import subprocess
import sys

import pytest

from paper_2412_07017_b200 import build as lib_build

HERE = os.path.dirname(os.path.abspath(__file__))


def run_child(*args):
    lib = lib_build.DEBUG_LIB
    inputs = lib_build.sources() + [os.path.join(lib_build.CSRC, f) for f in os.listdir(lib_build.CSRC)
                                    if f.endswith((".cuh", ".h"))]
    if not os.path.exists(lib) or any(os.path.getmtime(f) > os.path.getmtime(lib) for f in inputs):
        lib = lib_build.build(debug=True)
    env = dict(os.environ, ASYNCLM_LIBRARY=lib)
    proc = subprocess.run([sys.executable, os.path.join(HERE, "checked_build_child.py"), *args], env=env,
                          capture_output=True, text=True, timeout=600)
    assert proc.returncode == 0, proc.stdout + proc.stderr
    return json.loads(proc.stdout.strip().splitlines()[-1])


@pytest.mark.gpu
def test_bad_page_ids_set_the_status_word_and_are_not_dereferenced():
    res = run_child()
    assert res == {"clean": 0, "bad_id_warp_body": 43, "bad_id_span_body": 42}, res


@pytest.mark.gpu
def test_a_bounded_wait_that_runs_out_is_reported_and_the_next_step_is_correct():
    """The checked build can leave out one hand-off of the span body (a K tile that is never announced).
    Nothing sets that barrier, so the waits behind it run out after their cycle budget (about a second);
    the kernel returns, the status word names the wait, and the next step on the same context matches
    the oracle.  No trap, no fault, no endless loop is involved."""
    res = run_child("wait")
    assert res["stalled_status"] in (11, 12, 21, 24, 26, 31), res
    assert 500.0 < res["stalled_ms"] < 5000.0, res      # the budget is 2e9 cycles
    assert res["next_status"] == 0 and res["next_ms"] < 50.0, res
