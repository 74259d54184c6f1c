"""Safety paths of the kernel that normal operation never takes, exercised without harming the device.

* A bounded wait that runs out: a test hook withholds the published threshold of one segment and shortens
  the wait bound, so the CTAs that wait for that threshold give up after a fraction of a millisecond.  The
  kernel must return by itself, report SIDCO_ST_TIMEOUT, and the same residual must work again after a
  state reset.  Nothing traps, nothing spins without a bound.
* The -DSIDCO_BOUNDS_CHECK build (every index into a caller or workspace buffer is range-checked on the
  device before use) runs the ragged and random cases and must report no violation while matching the oracle.
"""
import os
import subprocess
import sys

import numpy as np
import pytest

from oracle import sidco_oracle as O
from paper_2101_10761_b200 import workloads as W
from parity_util import GpuRun, check_parity, f32

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)


@pytest.mark.parametrize("sid,max_stages", [(0, -1), (2, -3)])
def test_bounded_wait_runs_out_and_the_context_survives(sid, max_stages):
    import torch
    from paper_2101_10761_b200 import binding as B
    sizes = [20000, 700]                   # segment 0 spans many CTA runs: the others wait for the fitting run
    off = W.offsets_from_sizes(sizes)
    d = int(off[-1])
    delta = f32(0.01)
    run = GpuRun(off)
    try:
        g = W.ragged_case(21, sizes, 1e-3)
        ora = O.sidco_compress(g, np.zeros(d, np.float32), off, delta, sid, max_stages)
        gpu = run.step(g, delta, sid, max_stages)
        check_parity(gpu, ora, off)
        res_o = ora.residual

        B.sidco_set_test_hooks(spin_limit=1000, drop_publication_seg=0)
        try:
            t0 = torch.cuda.Event(enable_timing=True)
            t1 = torch.cuda.Event(enable_timing=True)
            t0.record()
            out = run.step(g, delta, sid, max_stages)           # returns: the waits are bounded
            t1.record()
            torch.cuda.synchronize()
        finally:
            B.sidco_set_test_hooks()                            # back to normal operation
        assert t0.elapsed_time(t1) < 2000.0
        assert all(sd.status & B.ST_TIMEOUT for sd in out["debug"]), "the time-out was not reported"
        # the results of such a call are invalid, but its count stays inside the buffers
        assert 0 <= int(out["out_k"][-1]) <= d

        # after a reset the same residual buffer behaves like a fresh one
        B.sidco_reset_state(run.res)
        res_o = np.zeros(d, np.float32)
        for call in range(3):
            g = W.ragged_case(30 + call, sizes, 1e-3)
            ora = O.sidco_compress(g, res_o, off, delta, sid, max_stages)
            gpu = run.step(g, delta, sid, max_stages)
            check_parity(gpu, ora, off)
            assert not any(sd.status & B.ST_TIMEOUT for sd in gpu["debug"])
            res_o = ora.residual
    finally:
        run.close()


CHECK_CODE = r'''
import sys, numpy as np
sys.path.insert(0, %r); sys.path.insert(0, %r)
from oracle import sidco_oracle as O
from paper_2101_10761_b200 import binding as B, workloads as W
from parity_util import GpuRun, check_parity, f32
assert B.sidco_build_flags() & B.BUILD_BOUNDS_CHECK
rng = np.random.Generator(np.random.PCG64(77))
cases = [([0, 1, 3, 31, 32, 33, 64, 1000, 8191, 8192, 8193, 20000], 0),
         ([5, 1023, 1025, 7, 40001, 2, 0, 300], 1), ([300000], 0), ([9, 70001, 13], 3)]
for _ in range(6):
    n = int(rng.integers(1, 40))
    cases.append(([int(x) for x in rng.integers(0, 30000, n)], int(rng.integers(0, 4))))
for sizes, shift in cases:
    off = W.offsets_from_sizes(sizes)
    d = int(off[-1])
    for sid, ms in ((0, 4), (1, -2), (2, -3), (0, -4)):
        run = GpuRun(off, base_shift=shift)
        res_o = np.zeros(d, np.float32)
        state = O.new_state(len(sizes))
        for call in range(6):
            g = W.ragged_case(100 + call, sizes, 1e-3)
            ora = O.sidco_compress(g, res_o, off, f32(0.01), sid, ms, state=state if ms > 0 else None)
            gpu = run.step(g, f32(0.01), sid, ms)
            check_parity(gpu, ora, off, state if ms > 0 else None)      # status must be equal: no violation bit
            res_o = ora.residual
        run.close()
print("bounds ok")
''' % (ROOT, HERE)


def test_bounds_checked_build_finds_no_violation():
    env = dict(os.environ, SIDCO_LIB_VARIANT="check")
    r = subprocess.run([sys.executable, "-c", CHECK_CODE], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "bounds ok" in r.stdout, (r.stdout[-1000:], r.stderr[-3000:])
