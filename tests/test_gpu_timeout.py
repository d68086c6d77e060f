"""The bounded device-side waits, made to run out.

Every wait in the expert kernels and in the cooperative selection kernel has a budget; when it is
spent the role raises the CTA's abort flag, writes the time-out status word, all roles leave, what
was started asynchronously is drained, TMEM is released and the kernel ends.  The shipped library
cannot be made to do that on demand, so a second build of the same sources (test hooks: budgets of
two milliseconds, and a switch under which the schedulers withhold their final "no more work"
message and the selection kernel's grid barrier expects one arrival too many) runs in a child
process.  Nothing faults, traps or spins without a bound.  Expected of every body: parity before,
MOEV_ETIMEOUT from moev_status_sync on the withheld call within a moment, the status word cleared,
parity on the two calls after it."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def child_result():
    from paper_2607_12696_b200.build import TEST_LIB, build
    build()
    assert os.path.exists(TEST_LIB)
    p = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "timeout_child.py")], capture_output=True,
                       text=True, timeout=600)
    assert p.returncode == 0, p.stdout[-2000:] + p.stderr[-4000:]
    line = [l for l in p.stdout.splitlines() if l.startswith("RESULT ")][-1]
    return json.loads(line[len("RESULT "):])


@pytest.mark.parametrize("body,impl", [("fp8_single_phase", 2), ("fp8_two_phase", 2), ("fp8_fold_scale", 2),
                                       ("bf16", 2), ("mxfp4", 2)])
def test_expert_kernel_wait_runs_out_and_context_stays_usable(child_result, body, impl):
    r = child_result[body]
    assert r["impl"] == impl                      # the tensor-core kernels (their waits are the bounded ones)
    assert r["timeout_status"] == 5               # MOEV_ETIMEOUT
    assert r["timeout_wall_s"] < 5.0              # budgets of milliseconds, not an unbounded spin
    assert r["status_after"] == 0                 # the read that reported it cleared the status word
    tol = 3e-2 if body == "mxfp4" else 1e-2
    assert r["err_before"] <= tol and r["err_after"] <= tol and r["err_after2"] <= tol


def test_selection_grid_barrier_runs_out(child_result):
    r = child_result["select_grid"]
    assert r["n_selected_withheld"] == -1
    assert r["timeout_wall_s"] < 5.0
    assert r["n_selected_after"] == 16 and r["selected_match"]
