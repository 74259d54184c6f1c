"""Pins for the CPU oracle: each check ties an oracle function to something the
paper or the mathematics fixes independently of the oracle's own code (closed
forms, library quantile functions, asymptotics on samples of a known law,
brute force on tiny inputs, scripted adaptation sequences)."""
import math
import os

import numpy as np
import pytest
import scipy.special as sps
import scipy.stats as sst

from oracle import sidco_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = float(line[1])
    return out


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def laplace_acc(n, b, seed):
    return rng(seed).laplace(0.0, b, n).astype(np.float32)


# ------------------------------------------------------------------ stage ratios

def test_stage_cap_values():
    # largest M with 0.25^(M-1) > delta
    assert O.stage_cap(0.1, 0.25) == 2
    assert O.stage_cap(0.01, 0.25) == 4
    assert O.stage_cap(0.001, 0.25) == 5
    assert O.stage_cap(0.25, 0.25) == 1
    assert O.stage_cap(0.5, 0.25) == 1


@pytest.mark.parametrize("delta", [0.1, 0.01, 0.001, 3e-4])
@pytest.mark.parametrize("M", [1, 2, 3, 4, 5])
def test_stage_ratios_product_is_delta(delta, M):
    M = min(M, O.stage_cap(delta, 0.25))
    r = O.stage_ratios(delta, M, 0.25)
    assert len(r) == M
    assert all(0.0 < x < 1.0 for x in r)
    assert math.prod(r) == pytest.approx(delta, rel=1e-14)
    assert all(x == 0.25 for x in r[:-1])


# ------------------------------------------------------------------ exponential

def test_exp_closed_form_golden():
    g = golden()
    assert O.exp_quantile_step(1e-3, 0.01) == pytest.approx(g["exp_eta_b1e-3_delta0.01"], rel=1e-14)
    assert O.exp_quantile_step(1e-3, 0.25) == pytest.approx(g["exp_eta1_b1e-3_delta0.25"], rel=1e-14)
    assert O.exp_quantile_step(1e-3, 0.04) == pytest.approx(g["exp_inc_b1e-3_delta0.04"], rel=1e-14)


def test_exp_threshold_is_library_quantile():
    # eta must be the (1-delta) quantile of Exp(scale = mean): library ppf.
    for mean, delta in [(0.3, 0.1), (2e-4, 0.001)]:
        assert O.exp_quantile_step(mean, delta) == pytest.approx(
            sst.expon(scale=mean).ppf(1.0 - delta), rel=1e-10)


def test_config1_single_stage_converges_to_b_log_inv_delta():
    g = golden()
    x = laplace_acc(262144, 1e-3, 0)
    res = O.sidco_compress(x, np.zeros_like(x), [0, x.size], 0.01, O.SID_EXP, -1)
    eta = res.report[0].eta[-1]
    # estimator std of the mean of n exponentials is b/sqrt(n)
    assert eta == pytest.approx(g["exp_eta_b1e-3_delta0.01"], rel=5 / math.sqrt(x.size))
    k = 0.01 * x.size
    assert abs(int(res.out_k[0]) - k) <= 5 * (50.9 + 23.6)


def test_config1_two_stage_memoryless():
    g = golden()
    x = laplace_acc(262144, 1e-3, 0)
    res = O.sidco_compress(x, np.zeros_like(x), [0, x.size], 0.01, O.SID_EXP, -2)
    rep = res.report[0]
    assert rep.M_used == 2
    assert rep.eta[0] == pytest.approx(g["exp_eta1_b1e-3_delta0.25"], rel=5 / math.sqrt(x.size))
    assert abs(rep.k_stage[0] - 65536) <= 5 * math.sqrt(x.size * 0.25 * 0.75) + 0.01 * 65536
    # the increment is fitted on ~65k exceedances
    assert rep.eta[1] - rep.eta[0] == pytest.approx(g["exp_inc_b1e-3_delta0.04"], rel=5 / math.sqrt(65536))
    assert rep.eta[1] == pytest.approx(g["exp_eta_b1e-3_delta0.01"], rel=0.02)


@pytest.mark.parametrize("M", [1, 2, 3, 4])
def test_exp_multistage_hits_target_ratio_on_exponential_data(M):
    # memorylessness: on Laplace data every stage count gives k/n -> delta
    n, delta = 400000, 0.01
    x = laplace_acc(n, 3e-2, 11)
    res = O.sidco_compress(x, np.zeros_like(x), [0, n], delta, O.SID_EXP, -M)
    k = delta * n
    assert abs(int(res.out_k[0]) - k) < 6 * math.sqrt(k) + 0.03 * k


# ------------------------------------------------------------------ GPD

def test_gpd_threshold_closed_form_golden_and_library():
    g = golden()
    a, b, delta = 0.2, 1.0, 0.01
    # population moments of GP(shape a, scale b)
    mean = b / (1 - a)
    var = b * b / ((1 - a) ** 2 * (1 - 2 * a))
    eta, deg = O.gpd_quantile_step(mean, var, delta)
    assert not deg
    assert eta == pytest.approx(g["gpd_eta_a0.2_b1_delta0.01"], rel=1e-12)
    assert eta == pytest.approx(sst.genpareto(c=a, scale=b).ppf(1 - delta), rel=1e-10)


@pytest.mark.parametrize("a,b", [(0.2, 1.0), (-0.2, 3.0), (0.05, 1e-3), (0.35, 0.1)])
@pytest.mark.parametrize("delta", [0.25, 0.01])
def test_gpd_moment_match_inverts_population_moments(a, b, delta):
    dist = sst.genpareto(c=a, scale=b)
    eta, _ = O.gpd_quantile_step(dist.mean(), dist.var(), delta)
    assert eta == pytest.approx(dist.ppf(1 - delta), rel=1e-9)


def test_gpd_alpha_to_zero_is_exponential():
    mean = 0.7
    eta, _ = O.gpd_quantile_step(mean, mean * mean, 0.01)      # R = 1 -> alpha = 0
    assert eta == pytest.approx(O.exp_quantile_step(mean, 0.01), rel=1e-12)
    eta2, _ = O.gpd_quantile_step(mean, mean * mean * (1 + 1e-9), 0.01)
    assert eta2 == pytest.approx(eta, rel=1e-7)


def test_gpd_zero_variance_is_limit_of_formula():
    mean = 2.5
    lim, deg = O.gpd_quantile_step(mean, 0.0, 0.01)
    assert deg and lim == mean
    near, _ = O.gpd_quantile_step(mean, mean * mean * 1e-9, 0.01)
    assert near == pytest.approx(lim, rel=1e-8)


def gp_sample(n, a, b, seed):
    u = rng(seed).random(n)
    x = (b / a) * np.expm1(-a * np.log1p(-u))          # inverse CDF of the paper's GPD
    sign = np.where(rng(seed + 1).random(n) < 0.5, -1.0, 1.0)
    return (sign * x).astype(np.float32)


@pytest.mark.parametrize("M", [1, 2, 3])
def test_gpd_on_gp_data_hits_target_ratio(M):
    # threshold stability of the GP family: every stage count should select ~delta*n
    n, delta = 1000000, 0.01
    x = gp_sample(n, 0.2, 1e-2, 5)
    res = O.sidco_compress(x, np.zeros_like(x), [0, n], delta, O.SID_GPD, -M)
    k = delta * n
    assert abs(int(res.out_k[0]) - k) < 6 * math.sqrt(k) + 0.10 * k
    eta = res.report[0].eta
    assert all(eta[i] < eta[i + 1] for i in range(len(eta) - 1))
    assert eta[-1] == pytest.approx(sst.genpareto(c=0.2, scale=1e-2).ppf(1 - delta), rel=0.06)


def test_gpd_on_exponential_data_matches_exp():
    n = 1000000
    x = laplace_acc(n, 1e-2, 6)
    r_g = O.sidco_compress(x, np.zeros_like(x), [0, n], 0.01, O.SID_GPD, -1).report[0]
    r_e = O.sidco_compress(x, np.zeros_like(x), [0, n], 0.01, O.SID_EXP, -1).report[0]
    assert r_g.eta[0] == pytest.approx(r_e.eta[0], rel=0.02)


# ------------------------------------------------------------------ gamma

@pytest.mark.parametrize("s", [1e-3, 0.05, 0.5772156649015329, 2.0, 9.0])
def test_gamma_shape_is_root_of_quadratic(s):
    al = O.gamma_shape(s)
    assert al > 0
    assert abs(6 * s * al * al - (3 - s) * al - 1) < 1e-10 * max(1.0, al * al * s)


def test_gamma_shape_at_euler_gamma_golden():
    assert O.gamma_shape(0.5772156649015329) == pytest.approx(
        golden()["gamma_shape_at_euler_gamma"], abs=5e-7)


@pytest.mark.parametrize("alpha,bias", [(0.2, -0.010), (0.4, -0.014), (0.6, -0.013), (1.0, -0.009), (2.0, -0.004)])
def test_gamma_shape_population_bias(alpha, bias):
    s = math.log(alpha) - sps.digamma(alpha)       # population value of log(mean) - mean(log)
    assert O.gamma_shape(s) / alpha - 1 == pytest.approx(bias, abs=1.5e-3)


def gamma_sample(n, alpha, theta, seed):
    r = rng(seed)
    return (np.where(r.random(n) < 0.5, -1.0, 1.0) * r.gamma(alpha, theta, n)).astype(np.float32)


@pytest.mark.parametrize("delta,expected", [(0.1, 0.66), (0.01, 0.50), (0.001, 0.42)])
def test_gamma_closed_form_underselects_gamma_data_by_the_known_factor(delta, expected):
    """On Gamma(0.6) magnitudes the closed-form threshold of Corollary 1.2 is an upper bound of the true
    quantile, so the single-stage gamma fit keeps fewer than k elements: the population values of
    k_hat / k are 0.66, 0.50 and 0.42 at delta = 0.1, 0.01, 0.001 (computed from the gamma survival function
    at the closed form evaluated with the biased shape estimate; independent of this oracle)."""
    n, alpha, theta = 2_000_000, 0.6, 2e-3
    x = gamma_sample(n, alpha, theta, 9)
    out = O.sidco_compress(x, np.zeros_like(x), [0, n], delta, O.SID_GAMMA, -1)
    ratio = out.idx.size / (delta * n)
    # population value recomputed here from library functions only
    s_pop = math.log(alpha) - sps.digamma(alpha)
    a_hat = (3 - s_pop + math.sqrt((s_pop - 3) ** 2 + 24 * s_pop)) / (12 * s_pop)
    eta_over_theta = -(alpha / a_hat) * (math.log(delta) + sps.gammaln(a_hat))
    pop = sst.gamma.sf(eta_over_theta, alpha) / delta
    assert pop == pytest.approx(expected, abs=0.01)
    k = delta * n
    assert ratio == pytest.approx(pop, abs=6 * math.sqrt(pop / k) + 0.02)


@pytest.mark.parametrize("alpha", [0.3, 0.6, 0.9])
@pytest.mark.parametrize("delta", [0.01, 0.001])
def test_gamma_threshold_of_the_oracle_upper_bounds_the_exact_quantile(alpha, delta):
    """Corollary 1.2: for a fitted shape <= 1 (and an exact quantile >= 1 in units of the scale) the closed form
    lies above beta * P^-1(alpha, 1 - delta).  Checked on the oracle's own output with a library inverse."""
    n = 300000
    x = gamma_sample(n, alpha, 1e-3, 31)
    a = np.abs(x).astype(np.float64)
    eta, deg = O.gamma_first_stage(a, delta)
    assert not deg
    s_hat = math.log(a.mean()) - np.log(a).mean()
    a_hat = O.gamma_shape(s_hat)
    b_hat = a.mean() / a_hat
    exact = sps.gammaincinv(a_hat, 1.0 - delta)
    assert a_hat <= 1.0 and exact >= 1.0
    assert eta / b_hat >= exact * (1 - 1e-12)
    # and the bound is tight at shape one (exponential data)
    e = np.abs(laplace_acc(n, 1e-3, 32)).astype(np.float64)
    eta1, _ = O.gamma_first_stage(e, delta)
    a1 = O.gamma_shape(math.log(e.mean()) - np.log(e).mean())
    assert eta1 / (e.mean() / a1) == pytest.approx(sps.gammaincinv(a1, 1.0 - delta), rel=0.02)


def test_gamma_on_exponential_data_close_to_exp_threshold():
    # exponential magnitudes are Gamma(1): shape -> 0.9909, threshold within a few % of b*ln(1/delta)
    n = 1000000
    x = laplace_acc(n, 1e-2, 12)
    rep = O.sidco_compress(x, np.zeros_like(x), [0, n], 0.01, O.SID_GAMMA, -1).report[0]
    assert rep.eta[0] == pytest.approx(1e-2 * math.log(100), rel=0.03)


def test_gamma_ignores_zeros_and_rescales_tail():
    # half the entries zero: the fit sees only nonzeros; tail prob becomes 2*delta among them
    n = 400000
    x = gamma_sample(n, 0.9, 1e-2, 21)
    z = np.concatenate([x, np.zeros(n, np.float32)])
    e_full, _ = O.gamma_first_stage(np.abs(z).astype(np.float64), 0.01)
    e_half, _ = O.gamma_first_stage(np.abs(x).astype(np.float64), 0.02)
    assert e_full == pytest.approx(e_half, rel=1e-12)


def test_gamma_clamp_and_constant_rules():
    # delta * Gamma(alpha_hat) >= 1 -> clamp to 0
    x = gamma_sample(200000, 0.05, 1.0, 3)
    eta, deg = O.gamma_first_stage(np.abs(x).astype(np.float64), 0.25)
    assert deg and eta == 0.0
    # constant magnitudes -> exponential formula
    c = np.full(1000, 0.125)
    eta, deg = O.gamma_first_stage(c, 0.01)
    assert deg and eta == pytest.approx(0.125 * math.log(100), rel=1e-12)


# ------------------------------------------------------------------ selection, residual, brute force

def brute_force_count(acc, eta):
    srt = sorted((abs(float(v)) for v in acc), reverse=True)
    c = 0
    for v in srt:
        if v >= eta:
            c += 1
        else:
            break
    return c


@pytest.mark.parametrize("n", [1, 3, 31, 32, 33, 64, 1000])
@pytest.mark.parametrize("sid", [O.SID_EXP, O.SID_GAMMA, O.SID_GPD])
@pytest.mark.parametrize("M", [1, 2, 3])
def test_selection_brute_force_tiny(n, sid, M):
    g = laplace_acc(n, 1e-2, 100 + n)
    r = laplace_acc(n, 3e-3, 200 + n)
    res = O.sidco_compress(g, r, [0, n], 0.1, sid, -M)
    acc = (g + r).astype(np.float32)
    assert np.array_equal(res.acc, acc)
    eta = res.report[0].eta[-1]
    assert int(res.out_k[0]) == brute_force_count(acc, eta) == res.idx.size
    assert np.all(np.diff(res.idx) > 0)
    assert np.array_equal(res.val, acc[res.idx])
    # residual + scatter(idx, val) == acc bit for bit, residual exactly zero on idx
    rebuilt = res.residual.copy()
    rebuilt[res.idx] += res.val
    assert np.array_equal(rebuilt, acc)
    assert np.all(res.residual[res.idx] == 0)
    mask = np.ones(n, bool)
    mask[res.idx] = False
    assert np.array_equal(res.residual[mask].view(np.uint32), acc[mask].view(np.uint32))
    # stage thresholds never decrease
    e = res.report[0].eta
    assert all(e[i] <= e[i + 1] for i in range(len(e) - 1))


def test_exceedance_counts_brute_force_each_stage():
    n = 500
    g = laplace_acc(n, 1.0, 77)
    res = O.sidco_compress(g, np.zeros_like(g), [0, n], 0.01, O.SID_GPD, -3)
    rep = res.report[0]
    mags = [abs(float(v)) for v in g]
    for m in range(rep.M_used - 1):
        assert rep.k_stage[m] == sum(1 for v in mags if v > rep.eta[m])
    assert rep.k_stage[-1] == sum(1 for v in mags if v >= rep.eta[-1])


def test_intermediate_exceedance_is_strict():
    # gamma first stage clamps to eta_1 = 0 here; the stage-2 exceedance set is |x| > 0
    # (strict, as in the stage loop of Algorithm 1), so exact zeros must not enter the refit
    x = np.concatenate([gamma_sample(200000, 0.05, 1.0, 3), np.zeros(1000, np.float32)])
    res = O.sidco_compress(x, np.zeros_like(x), [0, x.size], 0.1, O.SID_GAMMA, -2)
    rep = res.report[0]
    assert rep.eta[0] == 0.0
    assert rep.k_stage[0] == sum(1 for v in x if v != 0.0)


def test_two_stage_exp_hand_example():
    # |x| = 1..8, delta = 0.125, delta_1 = 0.25: eta_1 = 4.5 ln 4 = 6.238..;
    # exceedances {7, 8}: mean shift = 7.5 - eta_1; delta_2 = 0.5
    x = np.array([1, -2, 3, -4, 5, -6, 7, -8], dtype=np.float32)
    res = O.sidco_compress(x, np.zeros_like(x), [0, 8], 0.125, O.SID_EXP, -2)
    eta1 = 4.5 * math.log(4.0)
    eta2 = eta1 + (7.5 - eta1) * math.log(2.0)
    assert res.report[0].eta[0] == pytest.approx(eta1, rel=1e-14)
    assert res.report[0].eta[1] == pytest.approx(eta2, rel=1e-14)
    assert res.report[0].k_stage == [2, 1]
    assert list(res.idx) == [7] and list(res.val) == [-8.0]


def test_binomial_achieved_ratio_per_segment():
    # k_hat ~ Binomial(n, delta) (+ estimator error) when the family is right
    sizes = [50000, 120000, 80000]
    off = np.concatenate([[0], np.cumsum(sizes)])
    r = rng(31)
    g = np.concatenate([r.laplace(0, b, n) for b, n in zip([1e-4, 1e-2, 1.0], sizes)]).astype(np.float32)
    res = O.sidco_compress(g, np.zeros_like(g), off, 0.01, O.SID_EXP, -1)
    for s, n in enumerate(sizes):
        k = 0.01 * n
        assert abs(int(res.out_k[s]) - k) < 5 * math.sqrt(k) + 5 * k * math.log(100) / math.sqrt(n)
    assert int(res.out_k[-1]) == res.idx.size == int(res.out_k[:-1].sum())
    # indices are segment-major ascending and fall in their segment
    bounds = np.cumsum(res.out_k[:-1])
    for s in range(3):
        part = res.idx[(bounds[s] - res.out_k[s]):bounds[s]]
        assert np.all((part >= off[s]) & (part < off[s + 1]))


def test_degenerate_segments():
    sizes = [0, 5, 7, 1, 6]
    off = np.concatenate([[0], np.cumsum(sizes)])
    g = np.zeros(19, np.float32)
    g[5:12] = 0.5 * np.array([1, -1, 1, -1, 1, -1, 1], np.float32)   # constant magnitude
    g[12] = 3.0                                                     # single element
    g[13:19] = [1, 2, np.nan, 4, 5, 6]                              # NaN segment
    for sid in (O.SID_EXP, O.SID_GAMMA, O.SID_GPD):
        res = O.sidco_compress(g, np.zeros_like(g), off, 0.1, sid, -2)
        assert res.out_k[0] == 0
        assert res.out_k[1] == 0 and res.report[1].status & O.ST_ALL_ZERO
        assert math.isinf(res.report[1].eta[-1])
        assert res.out_k[4] == 0 and res.report[4].status & O.ST_NONFINITE
    res = O.sidco_compress(g, np.zeros_like(g), off, 0.1, O.SID_GPD, -1)
    # zero variance -> eta = mean -> ties at the threshold are all selected (>=)
    assert res.report[2].eta[0] == 0.5 and res.out_k[2] == 7
    assert res.report[3].eta[0] == 3.0 and res.out_k[3] == 1


# ------------------------------------------------------------------ adaptation

def test_adapt_stages_transition_table():
    k, eH, eL = 100.0, 0.2, 0.2
    assert O.adapt_stages(2, 121.0, k, eH, eL, 4) == 1      # too many -> fewer stages
    assert O.adapt_stages(2, 79.0, k, eH, eL, 4) == 3       # too few -> more stages
    assert O.adapt_stages(2, 120.0, k, eH, eL, 4) == 2      # boundary values stay
    assert O.adapt_stages(2, 80.0, k, eH, eL, 4) == 2
    assert O.adapt_stages(1, 500.0, k, eH, eL, 4) == 1      # clamped below
    assert O.adapt_stages(4, 1.0, k, eH, eL, 4) == 4        # clamped above


def test_adapt_update_scripted_sequence():
    p = O.Params()
    st = O.SegState()
    k = 100.0
    history = []
    script = [50] * 5 + [100] * 5 + [300] * 5 + [50, 50, 50, 50, 350]
    for kh in script:
        O.adapt_update(st, kh, k, p, 3)
        history.append(st.M)
    # changes only at calls 5, 10, 15, 20 and by at most one
    assert history[:4] == [1] * 4 and history[4] == 2
    assert history[5:10] == [2] * 5                      # mean 100 within tolerance
    assert history[10:14] == [2] * 4 and history[14] == 1
    assert history[19] == 1                              # mean 110 within tolerance
    assert st.k_sum == 0 and st.calls == 20


def test_adaptive_compress_moves_M_on_misfit_data():
    # Gamma(0.6) magnitudes with the gamma SID under-select at delta = 0.001 -> M grows
    n = 300000
    state = O.new_state(1)
    used = []
    for call in range(10):
        g = gamma_sample(n, 0.6, 1e-3, 500 + call)
        res = O.sidco_compress(g, np.zeros_like(g), [0, n], 0.001, O.SID_GAMMA, 4, state=state)
        used.append(res.report[0].M_used)
    assert used[:5] == [1] * 5
    assert used[5] == 2
    assert all(1 <= m <= 4 for m in used)
    assert all(abs(used[i + 1] - used[i]) <= 1 for i in range(9))


# ------------------------------------------------------------------ invariants

@pytest.mark.parametrize("sid", [O.SID_EXP, O.SID_GAMMA, O.SID_GPD])
@pytest.mark.parametrize("M", [1, 2, 3])
@pytest.mark.parametrize("k", [-20, 7])
def test_scale_equivariance(sid, M, k):
    # every fit is scale-equivariant: multiplying the data by 2^k (exact in floating point) multiplies
    # every threshold by 2^k and selects the same positions
    n = 50000
    x = gamma_sample(n, 0.7, 1e-2, 900 + M)
    r = laplace_acc(n, 1e-3, 901)
    a = O.sidco_compress(x, r, [0, 20000, n], 0.01, sid, -M)
    sc = np.float32(2.0 ** k)
    b = O.sidco_compress(x * sc, r * sc, [0, 20000, n], 0.01, sid, -M)
    assert np.array_equal(a.idx, b.idx)
    assert np.array_equal(a.val * sc, b.val)
    for ra, rb in zip(a.report, b.report):
        for ea, eb in zip(ra.eta, rb.eta):
            assert eb == pytest.approx(ea * 2.0 ** k, rel=1e-12)
        assert ra.k_stage == rb.k_stage


@pytest.mark.parametrize("sid", [O.SID_EXP, O.SID_GAMMA, O.SID_GPD])
def test_permutation_invariance_within_a_segment(sid):
    # thresholds depend on the multiset of magnitudes only; the selected values are the same multiset
    n = 30000
    x = gamma_sample(n, 0.5, 1.0, 950)
    perm = rng(951).permutation(n)
    a = O.sidco_compress(x, np.zeros_like(x), [0, n], 0.01, sid, -3)
    b = O.sidco_compress(x[perm], np.zeros_like(x), [0, n], 0.01, sid, -3)
    for ea, eb in zip(a.report[0].eta, b.report[0].eta):
        assert eb == pytest.approx(ea, rel=1e-12)
    assert a.report[0].k_stage == b.report[0].k_stage
    assert np.array_equal(np.sort(a.val), np.sort(b.val))
    assert np.array_equal(np.sort(perm[b.idx]), a.idx)


def test_sign_symmetry():
    # the model is symmetric around zero: flipping signs changes nothing but the signs of the values
    n = 20000
    x = laplace_acc(n, 1e-2, 960)
    a = O.sidco_compress(x, np.zeros_like(x), [0, n], 0.01, O.SID_GPD, -2)
    b = O.sidco_compress(-x, np.zeros_like(x), [0, n], 0.01, O.SID_GPD, -2)
    assert np.array_equal(a.idx, b.idx) and np.array_equal(a.val, -b.val)
    assert a.report[0].eta == b.report[0].eta


# ------------------------------------------------------------------ bf16 gradients

def test_bf16_widening_matches_an_independent_conversion():
    import torch
    r = rng(404)
    bits = r.integers(0, 1 << 16, 20000).astype(np.uint16)
    bits = bits[((bits >> 7) & 0xFF) != 0xFF]                 # finite values only (NaN payloads compare unequal)
    want = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    got = O.bf16_bits_to_f32(bits)
    assert got.dtype == np.float32 and np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # and rounding an fp32 to bf16 and back changes it by at most half a bf16 ulp
    x = r.standard_normal(1000).astype(np.float32)
    xb = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.all(np.abs(O.bf16_bits_to_f32(xb) - x) <= np.abs(x) * 2.0 ** -8)


# ------------------------------------------------------------------ variants the paper describes and replaces

@pytest.mark.parametrize("x", [0.03, 0.2, 0.6, 1.0, 2.5, 7.9, 8.0, 33.0, 400.0])
def test_digamma_and_trigamma_against_the_library(x):
    assert O.digamma(x) == pytest.approx(sps.digamma(x), rel=1e-12, abs=1e-12)
    assert O.trigamma(x) == pytest.approx(float(sps.polygamma(1, x)), rel=1e-10)


@pytest.mark.parametrize("a", [0.05, 0.3, 0.6, 1.0, 2.0, 9.0])
@pytest.mark.parametrize("q", [1.0, 0.9, 0.25, 0.04, 1e-3, 1e-7])
def test_gamma_upper_quantile_against_the_library_inverse(a, q):
    x = O.gamma_upper_quantile(a, q)
    if q >= 1.0:
        assert x == 0.0
        return
    assert x == pytest.approx(sps.gammainccinv(a, q), rel=1e-10)
    assert O.gamma_upper_q(a, x) == pytest.approx(q, rel=1e-10)
    assert O.gamma_upper_q(a, x) == pytest.approx(sps.gammaincc(a, x), rel=1e-11)


@pytest.mark.parametrize("s", [1e-3, 0.05, 0.5772156649, 1.5, 6.0])
def test_mle_shape_solves_the_digamma_equation(s):
    al = O.gamma_shape_mle(s)
    assert math.log(al) - sps.digamma(al) == pytest.approx(s, rel=1e-10, abs=1e-12)
    # Minka's closed form is within about 1.5 % of it
    assert O.gamma_shape(s) == pytest.approx(al, rel=0.02)


@pytest.mark.parametrize("alpha", [0.3, 0.6, 1.0, 2.0])
@pytest.mark.parametrize("delta", [0.1, 0.01, 0.001])
def test_exact_gamma_policy_reaches_the_target_ratio_on_gamma_data(alpha, delta):
    """With the maximum-likelihood shape and the exact quantile the single-stage gamma fit keeps k elements up
    to sampling error (binomial count plus the estimator's own error), where the closed form keeps 0.4-0.7 k."""
    n = 1_000_000
    x = gamma_sample(n, alpha, 2e-3, 40)
    pol = O.Policy(gamma_exact=True)
    out = O.sidco_compress(x, np.zeros_like(x), [0, n], delta, O.SID_GAMMA, -1, policy=pol)
    k = delta * n
    assert out.idx.size == pytest.approx(k, abs=6 * math.sqrt(k) + 0.03 * k)
    # the threshold is the library's quantile of the fitted law
    a = np.abs(x).astype(np.float64)
    s_hat = math.log(a.mean()) - np.log(a).mean()
    al = O.gamma_shape_mle(s_hat)
    assert out.report[0].eta[0] == pytest.approx(sst.gamma.isf(delta, al, scale=a.mean() / al), rel=1e-9)


def test_ratio_from_counts_policy_uses_the_achieved_count_of_the_previous_stage():
    n, delta = 400000, 0.001
    x = laplace_acc(n, 1e-3, 50)
    a = np.abs(x).astype(np.float64)
    pol = O.Policy(ratio_from_counts=True)
    for M in (2, 3, 4):
        rep_n = O.thresholds(a, delta, O.SID_EXP, M, 0.25)
        rep_c = O.thresholds(a, delta, O.SID_EXP, M, 0.25, pol)
        assert rep_c.eta[:-1] == rep_n.eta[:-1]                      # only the last stage changes
        exceed = a[a > rep_c.eta[-2]]
        want = rep_c.eta[-2] + (exceed - rep_c.eta[-2]).mean() * math.log(exceed.size / (delta * n))
        assert rep_c.eta[-1] == pytest.approx(want, rel=1e-12)
    # exponential magnitudes: the stages before the last keep a quarter each up to sampling error, so the two
    # rules nearly coincide, and both land on k
    k = delta * n
    for rep in (O.thresholds(a, delta, O.SID_EXP, 3, 0.25), O.thresholds(a, delta, O.SID_EXP, 3, 0.25, pol)):
        assert rep.k_stage[-1] == pytest.approx(k, abs=6 * math.sqrt(k) + 0.05 * k)


def test_reversed_adaptation_policy_flips_the_transition_table():
    for k_avg in (50.0, 100.0, 150.0):         # away from the clamps the two directions mirror each other
        fwd = O.adapt_stages(3, k_avg, 100.0, 0.2, 0.2, 5)
        rev = O.adapt_stages(3, k_avg, 100.0, 0.2, 0.2, 5, True)
        assert fwd - 3 == -(rev - 3)
    assert O.adapt_stages(2, 150.0, 100.0, 0.2, 0.2, 4, True) == 3        # too many -> one more stage
    assert O.adapt_stages(2, 50.0, 100.0, 0.2, 0.2, 4, True) == 1         # too few  -> one fewer
    assert O.adapt_stages(2, 110.0, 100.0, 0.2, 0.2, 4, True) == 2
    assert O.adapt_stages(1, 50.0, 100.0, 0.2, 0.2, 4, True) == 1 and O.adapt_stages(4, 150.0, 100.0, 0.2, 0.2, 4, True) == 4
    # scripted counts through the bookkeeping: five calls that select twice the target
    st_a, st_b = O.SegState(M=2), O.SegState(M=2)
    for _ in range(5):
        O.adapt_update(st_a, 200, 100.0, O.Params(), 4)
        O.adapt_update(st_b, 200, 100.0, O.Params(), 4, O.Policy(adapt_reversed=True))
    assert (st_a.M, st_a.calls, st_a.k_sum) == (1, 5, 0) and (st_b.M, st_b.calls, st_b.k_sum) == (3, 5, 0)
