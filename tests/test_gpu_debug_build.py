"""The bounds-checked build (-DSK_DEBUG=1) in place of a memory sanitizer.

Its kernels compare every hashed table offset, coordinate index, list position, histogram bin and shared-memory
window offset with the size of what it addresses; a violation is recorded in the handle's status word (reported by
sk_sync) and the access is skipped.  Here the small, odd-sized and multi-path cases of the parity suite run under
that build in a child process (the library is chosen when the binding is imported): they must stay parity-green AND
leave the status word at zero, since every step of them ends in sk_sync.  A second child checks the reporting path
itself with a check that is made to fail without any access behind it.
"""
import os
import subprocess
import sys

import pytest

from conftest import ROOT

pytestmark = pytest.mark.gpu


def _debug_env():
    from paper_2210_07454_b200 import build
    return dict(os.environ, SKETCHED_AMSGRAD_LIB=build.build(debug=True))


def test_small_and_odd_cases_run_clean_under_the_bounds_checked_build():
    env = _debug_env()
    select = ("edge or windowed or second_round or other_group_sizes or integer or scalar or checkpoint or flags "
              "or sketch_of_the_worker_sum or uneven or pa_")
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
                        "tests/test_gpu_parity.py", "tests/test_gpu_partitioned.py", "-k", select],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=2400)
    assert r.returncode == 0, r.stdout[-4000:] + r.stderr[-2000:]
    assert " passed" in r.stdout


CHILD = r"""
import numpy as np, torch
from paper_2210_07454_b200 import binding, synthetic
w = synthetic.WORKLOADS["C1"]
src = synthetic.GradientSource(w, device="cuda")
opt = binding.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k)
x = src.x0()
opt.step(src.grads(1), x); opt.sync()
I1 = opt.get("I")
for kind in (1, 2, 3, 4, 5, 6):
    opt.debug_check(kind)                       # a failed check of this kind, with no access behind it
    try:
        opt.sync()
    except binding.SkError as err:
        assert "status word = 0x%x" % (1 << kind) in str(err), str(err)
    else:
        raise SystemExit("the violation was not reported")
    opt.sync()                                  # reported once, then cleared: the handle stays usable
opt.step(src.grads(2), x); opt.sync()
assert len(opt.get("I")) == w.k and opt.stats()["status"] == 0.0
# a non-finite gradient entry is an invalid input: the debug build's kernels notice it and the host gets an error
fresh = binding.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k)
bad = src.grads(3).clone(); bad[1, 12345] = float("nan")
fresh.step(bad, src.x0())
try:
    fresh.sync()
except binding.SkError as err:
    assert "0x40" in str(err), str(err)
else:
    raise SystemExit("the non-finite entry was not reported")
print("child ok")
"""


def test_a_recorded_violation_reaches_the_host_and_the_handle_stays_usable():
    r = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=_debug_env(), capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "child ok" in r.stdout, r.stdout[-2000:] + r.stderr[-3000:]
