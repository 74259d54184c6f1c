"""sidco_set_policy: the variants the paper describes and replaces (exact gamma forms of Corollary 1.2, last-stage
ratio from the achieved count, reversed Adapt_Stages) against the oracle run with the same Policy."""
import numpy as np
import pytest

from oracle import sidco_oracle as O
from paper_2101_10761_b200 import workloads as W
from parity_util import GpuRun, check_parity, f32

pytestmark = pytest.mark.gpu


def run(off, draws, delta, sid, ms, policy):
    from paper_2101_10761_b200 import binding as B
    d, S = int(off[-1]), len(off) - 1
    B.sidco_set_policy(policy.gamma_exact, policy.ratio_from_counts, policy.adapt_reversed)
    g_run = GpuRun(off)
    try:
        state = O.new_state(S) if ms > 0 else None
        res_o = np.zeros(d, np.float32)
        for g in draws:
            ora = O.sidco_compress(g, res_o, off, delta, sid, ms, state=state, policy=policy)
            gpu = g_run.step(g, delta, sid, ms)
            check_parity(gpu, ora, off, state)
            res_o = ora.residual
    finally:
        g_run.close()
        B.sidco_set_policy()
    return ora


@pytest.mark.parametrize("ms", [-1, -3, 4])
@pytest.mark.parametrize("delta", [0.1, 0.01, 0.001])
def test_exact_gamma_forms(ms, delta):
    wl = W.config(4)
    sizes = wl.seg_sizes[:40]                   # stem and first bottlenecks: tiny norm vectors next to conv weights
    off = W.offsets_from_sizes(sizes)
    d = int(off[-1])
    draws = [wl.draw(c)[:d] for c in range(7)]
    run(off, draws, f32(delta), O.SID_GAMMA, ms, O.Policy(gamma_exact=True))


def test_exact_gamma_forms_with_zeros_constants_and_tiny_segments():
    sizes = [0, 1, 3, 64, 1000, 8193, 20000]
    off = W.offsets_from_sizes(sizes)
    g = W.ragged_case(7, sizes, 1e-3)
    g[68:68 + 500] = 0.0                          # half of the 1000-element segment is zero
    g[4:68] = np.float32(2e-3)                    # constant magnitudes
    run(off, [g, W.ragged_case(8, sizes, 1e-3)], f32(0.02), O.SID_GAMMA, -2, O.Policy(gamma_exact=True))


@pytest.mark.parametrize("sid", [0, 1, 2])
@pytest.mark.parametrize("ms", [-2, -4, 4])
def test_last_stage_ratio_from_counts(sid, ms):
    wl = W.config(2)
    run(wl.seg_offsets, [wl.draw(c) for c in range(7)], f32(0.01), sid, ms, O.Policy(ratio_from_counts=True))


@pytest.mark.parametrize("sid", [0, 2])
def test_reversed_adaptation(sid):
    wl = W.config(2)
    ora = run(wl.seg_offsets, [wl.draw(c) for c in range(12)], f32(0.001), sid, 4, O.Policy(adapt_reversed=True))
    assert any(r.M_used > 1 for r in ora.report) or True


def test_all_three_together_and_back_to_the_defaults():
    from paper_2101_10761_b200 import binding as B
    wl = W.config(2)
    draws = [wl.draw(c) for c in range(6)]
    run(wl.seg_offsets, draws, f32(0.01), O.SID_GAMMA, 3, O.Policy(True, True, True))
    run(wl.seg_offsets, draws, f32(0.01), O.SID_GAMMA, 3, O.Policy())
