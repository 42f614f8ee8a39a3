"""The bounds-checking build (-DRF_BOUNDS_CHECK) on the GPU.

With the toolkit's memory checker unavailable, this build is the evidence that the kernels index inside their arrays:
every global-memory write and every schedule read is checked on the device, a violation is reported through
dev_status as RF_ERR_BOUNDS and the access is skipped (nothing traps).  The small parity tests run once against it
in a child process (the library is chosen at load time), and must pass with the status word still 0; a schedule
whose counts are wrong is then handed to the checked attention kernel, which must refuse it with RF_ERR_BOUNDS and
leave the output untouched."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
import numpy as np, torch
sys.path.insert(0, {root!r}); sys.path.insert(0, {tests!r})
from paper_2505_21036_b200 import api, synth
import gpu_util as gu
assert api.load().rf_bounds_checked() == 1
wl = synth.small_workload("mid", H=4, D=128, T=6, fh=12, fw=11, L=37, wf=1, ws=20)
run = gu.Run(wl)
run.force_classes([0, 1, 2, 3])
run.build()
O, lse = run.sparse()                       # a correct schedule: status stays 0 (asserted inside)
run.sched.count.fill_(run.sched.nKmax + 7)  # a schedule that was not built for this shape
o, l = run.outputs()
api.rf_sparse_attn_fwd(run.shape, run.params, run.q, run.k, run.v, run.head_class, run.sched, o, l, run.ws, run.status)
torch.cuda.synchronize()
assert int(run.status.item()) == 7, int(run.status.item())     # RF_ERR_BOUNDS
assert bool(torch.isnan(o.float()).all())                       # the lists were not walked, nothing was written
run.mem.check("checked attention with a bad schedule")
print("bounds-check child ok")
"""


@pytest.fixture(scope="module")
def checked_lib():
    from paper_2505_21036_b200 import build
    return build.build(checked=True)


def run_child(args, lib, timeout=1200):
    env = dict(os.environ, RAINFUSION_LIBRARY=lib)
    return subprocess.run(args, env=env, cwd=ROOT, capture_output=True, text=True, timeout=timeout)


def test_small_parity_tests_pass_on_the_checked_build(checked_lib):
    r = run_child([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
                   "tests/test_gpu_parity.py", "tests/test_gpu_plus.py", "tests/test_golden.py", "tests/test_zz_no_alloc.py"], checked_lib)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]


def test_a_schedule_with_wrong_counts_is_refused_not_walked(checked_lib):
    code = CHILD.format(root=ROOT, tests=os.path.join(ROOT, "tests"))
    r = run_child([sys.executable, "-c", code], checked_lib, timeout=300)
    assert r.returncode == 0 and "bounds-check child ok" in r.stdout, r.stdout[-2000:] + r.stderr[-3000:]
