"""GPU tests of the remaining C-ABI entry points: host-buffer path, caller-owned workspace, adaptation
state checkpointing, Algorithm 1's constants, diagnostics."""
import numpy as np
import pytest

from oracle import sidco_oracle as O
from paper_2101_10761_b200 import workloads as W
from parity_util import GpuRun, check_parity, f32

pytestmark = pytest.mark.gpu


def test_host_buffer_entry_matches_oracle_over_several_calls():
    import torch
    from paper_2101_10761_b200 import binding as B
    wl = W.config(2)
    off, d, S = wl.seg_offsets, wl.d, wl.n_segs
    delta = f32(0.01)
    h_res = torch.zeros(d, dtype=torch.float32).pin_memory()
    h_idx = torch.empty(d, dtype=torch.int32).pin_memory()
    h_val = torch.empty(d, dtype=torch.float32).pin_memory()
    h_k = torch.zeros(S + 1, dtype=torch.int32).pin_memory()
    state = O.new_state(S)
    res_o = np.zeros(d, np.float32)
    try:
        for call in range(6):
            g = wl.draw(call)
            h_g = torch.from_numpy(g).pin_memory()
            B.sidco_compress_host(h_g, h_res, off, delta, B.SID_GPD, 3, h_idx, h_val, h_k)
            ora = O.sidco_compress(g, res_o, off, delta, O.SID_GPD, 3, state=state)
            res_o = ora.residual
            k = int(h_k[S])
            assert np.array_equal(h_k.numpy(), ora.out_k)
            assert np.array_equal(h_idx[:k].numpy(), ora.idx)
            assert np.array_equal(h_val[:k].numpy().view(np.uint32), ora.val.view(np.uint32))
            assert np.array_equal(h_res.numpy().view(np.uint32), ora.residual.view(np.uint32))
    finally:
        B.sidco_release(h_res)


def test_pageable_numpy_buffers_work_too():
    from paper_2101_10761_b200 import binding as B
    n = 5000
    g = W.ragged_case(3, [n], 1e-2)
    res = np.zeros(n, np.float32)
    idx = np.empty(n, np.int32)
    val = np.empty(n, np.float32)
    k = np.zeros(2, np.int32)
    try:
        B.sidco_compress_host(g, res, [0, n], f32(0.05), B.SID_EXP, -1, idx, val, k)
    finally:
        B.sidco_release(res)
    ora = O.sidco_compress(g, np.zeros(n, np.float32), [0, n], f32(0.05), O.SID_EXP, -1)
    assert np.array_equal(k, ora.out_k) and np.array_equal(idx[:k[1]], ora.idx)
    assert np.array_equal(res, ora.residual)


def test_caller_owned_workspace():
    import torch
    from paper_2101_10761_b200 import binding as B
    sizes = [7000, 123, 40000]
    off = W.offsets_from_sizes(sizes)
    d = int(off[-1])
    need = B.sidco_workspace_bytes(d, len(sizes))
    assert need > 8 * d
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda:0")
    base = (ws.data_ptr() + 255) // 256 * 256
    run = GpuRun(off)
    try:
        with pytest.raises(B.SidcoError) as err:
            B.sidco_set_workspace(run.res, base + 8, need)          # misaligned
        assert err.value.code == -8
        B.sidco_set_workspace(run.res, base, need)
        g = W.ragged_case(11, sizes, 1e-3)
        ora = O.sidco_compress(g, np.zeros(d, np.float32), off, f32(0.01), O.SID_GAMMA, -2)
        gpu = run.step(g, f32(0.01), O.SID_GAMMA, -2)
        check_parity(gpu, ora, off)
        with pytest.raises(B.SidcoError) as err:
            B.sidco_set_workspace(run.res, base, need)              # too late: already in use
        assert err.value.code == -8
    finally:
        run.close()
    small = torch.empty(4096, dtype=torch.uint8, device="cuda:0")
    run2 = GpuRun(off)
    try:
        B.sidco_set_workspace(run2.res, (small.data_ptr() + 255) // 256 * 256, 1024)
        with pytest.raises(B.SidcoError):
            run2.step(W.ragged_case(12, sizes, 1e-3), f32(0.01), O.SID_EXP, -1)   # workspace too small
    finally:
        B.sidco_release(run2.res)


def test_state_save_load_resumes_adaptation():
    """A run interrupted after 7 calls and resumed from the saved (M, calls, k_sum) blob continues exactly
    like the uninterrupted oracle run."""
    from paper_2101_10761_b200 import binding as B
    wl = W.config(2)
    off, S = wl.seg_offsets, wl.n_segs
    delta = f32(0.001)
    state = O.new_state(S)
    res_o = np.zeros(wl.d, np.float32)
    run = GpuRun(off)
    try:
        for call in range(7):
            ora = O.sidco_compress(wl.draw(call), res_o, off, delta, O.SID_GAMMA, 4, state=state)
            gpu = run.step(wl.draw(call), delta, O.SID_GAMMA, 4)
            check_parity(gpu, ora, off, state)
            res_o = ora.residual
        blob = B.sidco_state_save(run.res, S)
        assert blob.reshape(S, 3)[:, 1].tolist() == [7] * S
        assert blob.reshape(S, 3)[:, 0].tolist() == [st.M for st in state]
        saved_residual = gpu["residual"]
    finally:
        run.close()
    run = GpuRun(off, residual0=saved_residual)
    try:
        gpu = run.step(wl.draw(7), delta, O.SID_GAMMA, 4)         # creates the state for this residual
        ora = None
        # rewind: load the checkpoint, restore the residual, replay call 7 and go on
        B.sidco_state_load(run.res, blob)
        import torch
        run.res.copy_(torch.from_numpy(saved_residual))
        for call in range(7, 12):
            ora = O.sidco_compress(wl.draw(call), res_o, off, delta, O.SID_GAMMA, 4, state=state)
            gpu = run.step(wl.draw(call), delta, O.SID_GAMMA, 4)
            check_parity(gpu, ora, off, state)
            res_o = ora.residual
        with pytest.raises(B.SidcoError):
            B.sidco_state_load(run.res, np.zeros(3 * S, np.int64))   # M = 0 is not a valid state
    finally:
        run.close()


def test_set_params_changes_ratios_tolerances_and_period():
    from paper_2101_10761_b200 import binding as B
    wl = W.config(2)
    off, S = wl.seg_offsets, wl.n_segs
    delta = f32(0.001)
    params = O.Params(delta1=0.5, eps_H=0.05, eps_L=0.4, Q=3)
    B.sidco_set_params(params.delta1, params.eps_H, params.eps_L, params.Q)
    try:
        state = O.new_state(S)
        res_o = np.zeros(wl.d, np.float32)
        run = GpuRun(off)
        try:
            for call in range(10):
                ora = O.sidco_compress(wl.draw(call), res_o, off, delta, O.SID_GPD, 5, state=state, params=params)
                gpu = run.step(wl.draw(call), delta, O.SID_GPD, 5)
                check_parity(gpu, ora, off, state)
                res_o = ora.residual
            assert state[0].calls == 10 and all(st.k_sum >= 0 for st in state)
        finally:
            run.close()
        # delta_1 = 0.5 changes every stage ratio of a fixed three-stage call (0.5, 0.5, delta / 0.25)
        run = GpuRun(off)
        try:
            g = wl.draw(30)
            ora = O.sidco_compress(g, np.zeros(wl.d, np.float32), off, delta, O.SID_EXP, -3, params=params)
            ref = O.sidco_compress(g, np.zeros(wl.d, np.float32), off, delta, O.SID_EXP, -3)
            assert ora.report[0].eta[0] != ref.report[0].eta[0]
            check_parity(run.step(g, delta, O.SID_EXP, -3), ora, off)
        finally:
            run.close()
    finally:
        B.sidco_set_params()          # back to the paper's settings
    with pytest.raises(B.SidcoError):
        B.sidco_set_params(delta1=0.0)


def test_diagnostics_and_bookkeeping():
    from paper_2101_10761_b200 import binding as B
    sizes = [300000]
    off = W.offsets_from_sizes(sizes)
    run = GpuRun(off)
    try:
        before = B.sidco_launch_count()
        run.step(W.ragged_case(5, sizes, 1e-3), f32(0.01), O.SID_EXP, -3)
        assert B.sidco_launch_count() == before + 1           # the whole call is one kernel
        # the product build takes no device timestamps: the profiling helpers say so
        assert B.sidco_build_flags() == 0
        with pytest.raises(B.SidcoError) as err:
            B.sidco_get_phase_times(run.res)
        assert err.value.code == -12
        with pytest.raises(B.SidcoError) as err:
            B.sidco_get_cta_sweep_times(run.res)
        assert err.value.code == -12
        B.sidco_reset_state_async(run.res)
        assert B.sidco_launch_count() == before + 2
    finally:
        run.close()
    with pytest.raises(B.SidcoError) as err:
        B.sidco_get_debug(run.res, 1)                          # released: no state for this pointer
    assert err.value.code == -7
    assert B.sidco_version() >= 200 and "delta" in B.sidco_error_string(-3)


def test_profile_build_reports_phase_times():
    """The -DSIDCO_PROFILE build of the same sources (loaded in a child process) stamps the phases."""
    import os
    import subprocess
    import sys
    code = r'''
import sys, numpy as np
sys.path.insert(0, %r); sys.path.insert(0, %r)
from paper_2101_10761_b200 import binding as B, workloads as W
from parity_util import GpuRun, f32
assert B.sidco_build_flags() & B.BUILD_PROFILE
sizes = [300000]
run = GpuRun(W.offsets_from_sizes(sizes))
run.step(W.ragged_case(5, sizes, 1e-3), f32(0.01), 0, -3)
ph = B.sidco_get_phase_times(run.res)
assert len(ph) == 12 and all(0.0 <= x < 1e5 for x in ph[:6]) and ph[5] >= ph[0] > 0, ph
ct = B.sidco_get_cta_sweep_times(run.res)
assert ct.shape[1] == 4 and ct.shape[0] >= 1 and np.all(ct[:, 0] > 0)
run.close()
print("profile ok")
''' % (os.path.dirname(os.path.dirname(os.path.abspath(__file__))), os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, SIDCO_LIB_VARIANT="profile")
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "profile ok" in r.stdout, (r.stdout[-1000:], r.stderr[-3000:])
