"""GPU-vs-oracle parity through the C ABI on the five benchmark configurations
and on edge cases.  Tolerances: thresholds within 1e-6 relative; indices
identical except inside the 1e-6*eta band; values and residual bit exact."""
import math

import numpy as np
import pytest

from oracle import sidco_oracle as O
from paper_2101_10761_b200 import workloads as W
from parity_util import GpuRun, check_parity, f32

pytestmark = pytest.mark.gpu

SIDS = [O.SID_EXP, O.SID_GAMMA, O.SID_GPD]


def run_sequence(wl_offsets, grads, delta, sid, max_stages, residual0=None, base_shift=0, check_status=True):
    """Feed the same gradients to both sides, carrying each side's own residual."""
    delta = f32(delta)
    off = np.asarray(wl_offsets, dtype=np.int64)
    d = int(off[-1])
    run = GpuRun(off, residual0, base_shift)
    res_o = np.zeros(d, np.float32) if residual0 is None else np.asarray(residual0, np.float32).copy()
    state = O.new_state(off.size - 1) if max_stages > 0 else None
    bands = 0
    try:
        for g in grads:
            ora = O.sidco_compress(g, res_o, off, delta, sid, max_stages, state=state)
            gpu = run.step(g, delta, sid, max_stages)
            b = check_parity(gpu, ora, off, state, check_status)
            bands += b
            # after a tolerated tie at the threshold both sides continue from the GPU's residual
            res_o = gpu["residual"] if b else ora.residual
    finally:
        run.close()
    return bands


# ------------------------------------------------------------------ config 1

@pytest.mark.parametrize("M", [1, 2])
def test_config1_laplace(M):
    wl = W.config(1)
    run_sequence(wl.seg_offsets, [wl.draw(0)], 0.01, O.SID_EXP, -M)


# ------------------------------------------------------------------ config 2

@pytest.mark.parametrize("sid", SIDS)
@pytest.mark.parametrize("delta", [0.1, 0.01, 0.001])
@pytest.mark.parametrize("max_stages", [-1, 4])
def test_config2_resnet20_shaped(sid, delta, max_stages):
    wl = W.config(2)
    # nonzero residual: what one prior (oracle) step leaves behind
    prior = O.sidco_compress(wl.draw(0), np.zeros(wl.d, np.float32), wl.seg_offsets, f32(delta), sid, -1)
    run_sequence(wl.seg_offsets, [wl.draw(1)], delta, sid, max_stages, residual0=prior.residual)


@pytest.mark.parametrize("sid", SIDS)
def test_config2_adaptive_many_calls(sid):
    wl = W.config(2)
    run_sequence(wl.seg_offsets, [wl.draw(c) for c in range(12)], 0.001, sid, 4)


# ------------------------------------------------------------------ config 3

@pytest.mark.parametrize("max_stages", [-3, 3])
def test_config3_vgg16_shaped(max_stages):
    wl = W.config(3)
    n = 1 if max_stages < 0 else 11
    run_sequence(wl.seg_offsets, [wl.draw(c) for c in range(n)], 0.001, O.SID_GPD, max_stages)


# ------------------------------------------------------------------ config 4 (full size, bench launch configuration)

@pytest.fixture(scope="module")
def config4_draws():
    wl = W.config(4)
    return wl, [wl.draw(c) for c in range(10)]


@pytest.mark.parametrize("sid", SIDS)
@pytest.mark.parametrize("delta", [0.01, 0.001])
def test_config4_resnet50_shaped_ten_calls(config4_draws, sid, delta):
    wl, draws = config4_draws
    run_sequence(wl.seg_offsets, draws, delta, sid, 4)


# ------------------------------------------------------------------ config 5

def test_config5_lstm_shaped_adaptive():
    wl = W.config(5)
    grads = (wl.draw(c) for c in range(11))
    run_sequence(wl.seg_offsets, grads, 0.001, O.SID_EXP, 4)


# ------------------------------------------------------------------ edge cases

@pytest.mark.parametrize("n", [0, 1, 3, 31, 32, 33, 64, 1000, 8191, 8192, 8193, 20000])
@pytest.mark.parametrize("sid", SIDS)
@pytest.mark.parametrize("M", [1, 3])
def test_single_segment_sizes(n, sid, M):
    g = W.ragged_case(50 + n, [n], 1e-2)
    r = W.ragged_case(90 + n, [n], 3e-3)
    run_sequence([0, n], [g], 0.1, sid, -M, residual0=r)


@pytest.mark.parametrize("sid", SIDS)
@pytest.mark.parametrize("base_shift", [0, 1, 2, 3, 4])
def test_unaligned_offsets_and_pointers(sid, base_shift):
    # offsets congruent to 1, 2, 3 (mod 4), empty segments, segments crossing tile windows
    sizes = [5, 0, 8190, 3, 0, 9001, 2, 16385, 1, 777, 0]
    off = W.offsets_from_sizes(sizes)
    g = [W.ragged_case(300 + c, sizes, 1e-3) for c in range(6)]
    run_sequence(off, g, 0.01, sid, 3, base_shift=base_shift)


@pytest.mark.parametrize("sid", SIDS)
@pytest.mark.parametrize("max_stages", [-1, 2])
def test_threshold_jumps_between_calls(sid, max_stages):
    """Single-stage segments pre-select candidates against a fraction of the previous call's threshold.
    Gradients that cancel the residual and shrink (or blow up) the scale by 1000x make the new
    threshold fall far below (or above) that guess; the output must not depend on it."""
    sizes = [30000, 5, 70001, 12000]
    off = W.offsets_from_sizes(sizes)
    d = int(off[-1])
    delta = f32(0.01)
    run = GpuRun(off)
    res_o = np.zeros(d, np.float32)
    state = O.new_state(len(sizes)) if max_stages > 0 else None
    scales = [1.0, 1e-3, 1e-3, 1.0, 1e3, 1e-3, 1.0]
    try:
        for call, sc in enumerate(scales):
            g = (sc * W.ragged_case(700 + call, sizes, 1e-2)).astype(np.float32)
            if call in (1, 5):
                g = (g - res_o).astype(np.float32)      # acc becomes the small fresh draw alone
            ora = O.sidco_compress(g, res_o, off, delta, sid, max_stages, state=state)
            gpu = run.step(g, delta, sid, max_stages)
            assert check_parity(gpu, ora, off, state) == 0
            res_o = ora.residual
    finally:
        run.close()


@pytest.mark.parametrize("sid", SIDS)
@pytest.mark.parametrize("M", [1, 2, 3])
def test_degenerate_segments(sid, M):
    sizes = [0, 5000, 7000, 1, 6, 3000]
    off = W.offsets_from_sizes(sizes)
    g = W.ragged_case(7, sizes, 1.0)
    g[off[1]:off[2]] = 0.0                                             # all-zero segment
    g[off[2]:off[3]] = 0.5 * np.where(np.arange(7000) % 2 == 0, 1, -1)  # constant magnitude
    g[off[3]] = 3.0                                                    # single element
    # last segment: half exact zeros
    seg = g[off[5]:off[6]]
    seg[::2] = 0.0
    run_sequence(off, [g], 0.05, sid, -M)


@pytest.mark.parametrize("sid", SIDS)
def test_nan_and_inf_segments_select_nothing(sid):
    import torch
    from paper_2101_10761_b200 import binding as B
    sizes = [4000, 4000, 4000]
    off = W.offsets_from_sizes(sizes)
    g = W.ragged_case(8, sizes, 1.0)
    g[4100] = np.nan
    g[8100] = np.inf
    run = GpuRun(off)
    try:
        out = run.step(g, f32(0.05), sid, -2)
    finally:
        run.close()
    ora = O.sidco_compress(g, np.zeros_like(g), off, f32(0.05), sid, -2)
    assert out["out_k"][1] == 0 and out["out_k"][2] == 0
    assert out["debug"][1].status & B.ST_NONFINITE and out["debug"][2].status & B.ST_NONFINITE
    assert math.isnan(out["debug"][1].eta[1]) and math.isnan(out["debug"][2].eta[1])
    assert np.array_equal(out["out_k"], ora.out_k)
    assert np.array_equal(out["idx"], ora.idx)
    assert np.array_equal(out["residual"], ora.residual, equal_nan=True)


def test_thresholds_independent_of_grid_size():
    """Deterministic two-level combine: the same input gives bit-identical thresholds whatever the
    number of CTAs (checked by running child processes with smaller grids)."""
    import json
    import os
    import subprocess
    import sys
    code = r'''
import json, sys, numpy as np, torch
sys.path.insert(0, %r); sys.path.insert(0, %r)
from paper_2101_10761_b200 import workloads as W
from parity_util import GpuRun, f32
wl = W.config(3)
run = GpuRun(wl.seg_offsets)
out = run.step(wl.draw(0), f32(0.001), 1, -3)
print(json.dumps([[d.eta[m].hex() for m in range(3)] for d in out["debug"]] + [out["idx"][:50].tolist(), int(out["out_k"][-1])]))
''' % (os.path.dirname(os.path.dirname(os.path.abspath(__file__))), os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for grid in ("100000", "37", "5"):
        env = dict(os.environ, SIDCO_GRID=grid)
        r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr[-2000:]
        outs.append(json.loads(r.stdout.strip().splitlines()[-1]))
    assert outs[0] == outs[1] == outs[2]


def test_giant_segments_are_summed_in_tiles_whatever_the_grid():
    """A segment of more than 4096 chunks is summed in two levels (tiles counted from the segment's first
    chunk).  Thresholds must match the oracle and be bit-identical for every grid."""
    import json
    import os
    import subprocess
    import sys
    code = r'''
import json, sys, numpy as np
sys.path.insert(0, %r); sys.path.insert(0, %r)
from oracle import sidco_oracle as O
from paper_2101_10761_b200 import workloads as W
from parity_util import GpuRun, check_parity, f32
sizes = [777, 6_000_123, 4_300_000, 50]
off = W.offsets_from_sizes(sizes)
run = GpuRun(off)
res_o = np.zeros(int(off[-1]), np.float32)
for call in range(2):
    g = W.ragged_case(300 + call, sizes, 1e-3)
    ora = O.sidco_compress(g, res_o, off, f32(0.001), 2, -3)
    out = run.step(g, f32(0.001), 2, -3)
    check_parity(out, ora, off)
    res_o = ora.residual
print(json.dumps([[d.eta[m].hex() for m in range(3)] for d in out["debug"]] + [int(out["out_k"][-1])]))
''' % (os.path.dirname(os.path.dirname(os.path.abspath(__file__))), os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for grid in ("100000", "37", "5"):
        env = dict(os.environ, SIDCO_GRID=grid)
        r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)
        assert r.returncode == 0, r.stderr[-3000:]
        outs.append(json.loads(r.stdout.strip().splitlines()[-1]))
    assert outs[0] == outs[1] == outs[2]


@pytest.mark.parametrize("mode", ["0", "2"])
def test_selection_routes_agree_with_the_oracle(mode):
    """The final selection has several routes (recorded candidate slots, listed chunks joined to them slot by slot,
    the warps' pass over chunks, the per-chunk staging).  Mode 0 records no candidates at all; mode 2 sets every
    candidate threshold too high, so that most recorded candidates are found unusable.  Both must reproduce the
    oracle over several calls, for one- and two-stage segments, ragged and tiny segments included."""
    import os
    import subprocess
    import sys
    code = r'''
import sys, numpy as np
sys.path.insert(0, %r); sys.path.insert(0, %r)
from oracle import sidco_oracle as O
from paper_2101_10761_b200 import workloads as W
from parity_util import GpuRun, check_parity, f32
sizes = [40_000, 64, 300_000, 7, 1024, 123_457, 2048, 16, 700_000, 33]
off = W.offsets_from_sizes(sizes)
for sid, ms, delta in ((0, 1, 0.001), (0, -2, 0.001), (2, 3, 0.01), (1, -2, 0.05)):
    run = GpuRun(off)
    res_o = np.zeros(int(off[-1]), np.float32)
    state = O.new_state(len(sizes))
    for call in range(4):
        g = W.ragged_case(900 + call, sizes, 1e-3)
        ora = O.sidco_compress(g, res_o, off, f32(delta), sid, ms, state=state)
        out = run.step(g, f32(delta), sid, ms)
        check_parity(out, ora, off)
        res_o = ora.residual
    run.close()
print("ok")
''' % (os.path.dirname(os.path.dirname(os.path.abspath(__file__))), os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, SIDCO_SPEC=mode)
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and r.stdout.strip().endswith("ok"), (r.stdout[-500:], r.stderr[-3000:])


@pytest.mark.parametrize("sid", SIDS)
@pytest.mark.parametrize("M", [2, 3])
def test_ties_with_the_first_threshold(sid, M):
    """Segments whose magnitudes are all equal (or that hold one element) make the moment-matched fit return
    eta_1 = the magnitude itself, no later stage raises it, and the rule |x| >= eta_M selects everything.  The
    elements equal to eta_1 are no exceedances, yet must reach the final selection.  Indices are compared
    exactly here (the usual tolerance band would hide a miss), over several calls."""
    sizes = [1, 4000, 7, 1, 2500, 3000]
    off = W.offsets_from_sizes(sizes)
    d = int(off[-1])
    run = GpuRun(off)
    res_o = np.zeros(d, np.float32)
    try:
        for call in range(3):
            g = W.ragged_case(40 + call, sizes, 1e-2)
            g[off[1]:off[2]] = np.float32(0.25) * np.where(np.arange(4000) % 3 == 0, -1, 1)     # equal magnitudes
            g[off[4]:off[5]] = np.float32(0.125 * (call + 1))
            ora = O.sidco_compress(g, res_o, off, f32(0.05), sid, -M)
            gpu = run.step(g, f32(0.05), sid, -M)
            check_parity(gpu, ora, off)
            assert np.array_equal(gpu["idx"], ora.idx), f"call {call}: index sets differ"
            assert np.array_equal(gpu["residual"].view(np.uint32), ora.residual.view(np.uint32))
            res_o = ora.residual
    finally:
        run.close()


@pytest.mark.parametrize("delta", [0.01, 0.03])
def test_many_survivors_per_run(delta):
    """About a thousand (delta = 0.01) or three thousand (0.03) survivors per CTA: around and above what a run keeps
    in shared memory for the placement, and more flagged slots than one round (0.01) or one pass (0.03) of the
    block-wide selection takes."""
    wl = W.config(3)
    off = wl.seg_offsets
    run = GpuRun(off)
    res_o = np.zeros(wl.d, np.float32)
    try:
        for call in range(3):
            g = wl.draw(call)
            ora = O.sidco_compress(g, res_o, off, f32(delta), O.SID_EXP, -1)
            gpu = run.step(g, f32(delta), O.SID_EXP, -1)
            check_parity(gpu, ora, off)
            res_o = ora.residual
    finally:
        run.close()


@pytest.mark.parametrize("sid,max_stages", [(0, -1), (2, -2)])
def test_long_runs_of_chunks_per_cta(sid, max_stages):
    """With three CTAs a run holds about 4800 chunks: the block-wide selection pass then needs several passes
    and does not cover the whole run, so the per-warp loop has to skip what the pass took.  Three calls, so
    that candidate flags exist from the second call on."""
    import os
    import subprocess
    import sys
    code = r'''
import sys, numpy as np
sys.path.insert(0, %r); sys.path.insert(0, %r)
from oracle import sidco_oracle as O
from paper_2101_10761_b200 import workloads as W
from parity_util import GpuRun, check_parity, f32
sid, ms = %d, %d
wl = W.config(3)
off, delta = wl.seg_offsets, f32(0.001)
run = GpuRun(off)
res_o = np.zeros(wl.d, np.float32)
for call in range(3):
    g = wl.draw(call)
    ora = O.sidco_compress(g, res_o, off, delta, sid, ms)
    gpu = run.step(g, delta, sid, ms)
    check_parity(gpu, ora, off)
    res_o = ora.residual
run.close()
print("parity ok")
''' % (os.path.dirname(os.path.dirname(os.path.abspath(__file__))), os.path.dirname(os.path.abspath(__file__)), sid, max_stages)
    env = dict(os.environ, SIDCO_GRID="3")
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "parity ok" in r.stdout, (r.stdout[-1000:], r.stderr[-3000:])


@pytest.mark.parametrize("use_async", [False, True])
def test_reset_declares_the_residual_empty(use_async):
    """After a reset the next call must behave as if the residual were all zeros, whatever it holds,
    and the adaptation must start again from M = 1."""
    import torch
    from paper_2101_10761_b200 import binding as B
    wl = W.config(2)
    off = wl.seg_offsets
    delta = f32(0.001)
    run = GpuRun(off)
    try:
        state = O.new_state(wl.n_segs)
        res_o = np.zeros(wl.d, np.float32)
        for call in range(7):                      # past one adaptation point, residual now non-zero
            ora = O.sidco_compress(wl.draw(call), res_o, off, delta, O.SID_GAMMA, 4, state=state)
            gpu = run.step(wl.draw(call), delta, O.SID_GAMMA, 4)
            check_parity(gpu, ora, off, state)
            res_o = ora.residual
        assert any(st.M > 1 for st in state)
        if use_async:
            B.sidco_reset_state_async(run.res)
        else:
            B.sidco_reset_state(run.res)
        state = O.new_state(wl.n_segs)
        res_o = np.zeros(wl.d, np.float32)         # the GPU buffer still holds the old residual
        for call in range(3):
            ora = O.sidco_compress(wl.draw(20 + call), res_o, off, delta, O.SID_GAMMA, 4, state=state)
            gpu = run.step(wl.draw(20 + call), delta, O.SID_GAMMA, 4)
            check_parity(gpu, ora, off, state)
            res_o = ora.residual
    finally:
        run.close()
