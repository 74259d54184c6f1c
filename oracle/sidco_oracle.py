"""CPU oracle for the SIDCo gradient sparsifier (test infrastructure only).

A plain, slow, fp64 restatement of the method, written from the paper's
equations and Algorithm 1 so that it can be checked against them by eye.  It
is NOT part of the product: only the tests, the smoke check and the benchmark's
CPU-baseline leg may import it, and it shares no code with the CUDA path.

What follows which passage
--------------------------
* error compensation ``acc = g + residual``: the memory-based update stated in
  the appendix on gradient distributions (one fp32 add per element);
* double-exponential fit and threshold: Corollary 1.1, Eq. (LaplaceThreshold);
* double-gamma fit and closed-form threshold: Corollary 1.2 (Minka's shape
  approximation, threshold from the bound on the incomplete gamma function);
* generalised-Pareto moment-matching fit and threshold: Corollary 1.3;
* peaks-over-threshold stages: Lemma 2 (GPD) and Corollary 2.1 (exponential),
  with the stage families stated after Corollary 2.1;
* threshold sparsification: the indicator definition in Section 2.3;
* stage-count adaptation: Algorithm 1, function Adapt_Stages.

Every floating-point step is fp64 except the error-compensation add, which is
the fp32 add the data path performs.  Where the paper is silent or garbled the
reading taken is marked ``[reading]`` and explained in the design document.

Pins (see tests): all functions here are pinned by closed forms, library
quantile functions, asymptotics on samples of known distributions, brute force
on tiny inputs and scripted adaptation sequences, except the numerical guards
for degenerate fits, which are "parity unpinned" beyond consistency checks.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

SID_EXP = 0
SID_GAMMA = 1
SID_GPD = 2

ST_NONFINITE = 1       # a magnitude in the segment is NaN or infinite
ST_DEGENERATE = 2      # a fit hit one of the degenerate-case rules
ST_ALL_ZERO = 4        # every magnitude in the segment is zero


@dataclass
class Params:
    """Constants of Algorithm 1 (defaults from the experimental settings)."""
    delta1: float = 0.25     # first-stage ratio
    eps_H: float = 0.2       # upper tolerance on the achieved count
    eps_L: float = 0.2       # lower tolerance
    Q: int = 5               # adaptation period in calls


@dataclass
class Policy:
    """Variants the paper describes and then replaces or leaves open.  All off: the method as evaluated.

    gamma_exact        Corollary 1.2 without its two shortcuts: the shape is the maximum-likelihood estimate
                       (root of the digamma equation the proof states) and the threshold is
                       beta * P^{-1}(alpha, 1 - delta), the exact quantile, instead of the closed-form bound.
    ratio_from_counts  the last stage aims at the target count directly: its ratio is k / k_hat_{M-1}
                       (target count over the exceedances the stage before it left) instead of the nominal
                       delta / delta_1^(M-1).  [reading: the paper only states delta = prod delta_m]
    adapt_reversed     Adapt_Stages with the opposite sign (too many selected -> one stage more), the
                       direction the prose of the experiments suggests; Algorithm 1 prints the other one.
    """
    gamma_exact: bool = False
    ratio_from_counts: bool = False
    adapt_reversed: bool = False


@dataclass
class SegState:
    """Adaptation state of one segment, carried across calls."""
    M: int = 1
    calls: int = 0
    k_sum: int = 0


@dataclass
class SegReport:
    M_used: int = 0
    eta: List[float] = field(default_factory=list)     # eta_1 .. eta_M_used
    k_stage: List[int] = field(default_factory=list)   # exceedances of each eta_m
    status: int = 0


@dataclass
class Result:
    idx: np.ndarray          # int32, ascending flat indices of the survivors
    val: np.ndarray          # float32, acc at those indices
    out_k: np.ndarray        # int32[n_segs + 1], per-segment counts then total
    residual: np.ndarray     # float32[d], acc with the survivors set to +0
    acc: np.ndarray          # float32[d], g + residual_in
    report: List[SegReport]


# ---------------------------------------------------------------------------
# Stage ratios
# ---------------------------------------------------------------------------

def stage_cap(delta: float, delta1: float) -> int:
    """Largest M with delta1**(M-1) > delta.  [reading] every non-final stage
    keeps a fraction delta1, the last one takes what is left, and there are
    never more stages than leave the last ratio below one."""
    M, p = 1, 1.0
    while True:
        p *= delta1
        if not (p > delta) or M >= 64:
            return M
        M += 1


def stage_ratios(delta: float, M: int, delta1: float) -> List[float]:
    """delta_1..delta_M with product delta (Section 2.4: delta = prod delta_m)."""
    if M == 1:
        return [delta]
    p = 1.0
    for _ in range(M - 1):
        p *= delta1
    return [delta1] * (M - 1) + [delta / p]


# ---------------------------------------------------------------------------
# Closed-form fits (Thresh_Estimation)
# ---------------------------------------------------------------------------

def gpd_quantile_step(mean: float, var: float, ratio: float):
    """Corollary 1.3 / Lemma 2: moment-matched GPD, threshold at tail
    probability ``ratio``.  Returns (eta, degenerate)."""
    if var == 0.0:
        # [reading] no spread: limit of the formula as mean^2/var -> infinity.
        return mean, True
    R = mean * mean / var
    alpha = 0.5 * (1.0 - R)
    beta = 0.5 * mean * (R + 1.0)
    t = -alpha * math.log(ratio)
    if abs(t) < 1e-12:
        # alpha -> 0: the GPD becomes the exponential distribution.
        return beta * math.log(1.0 / ratio), False
    return (beta / alpha) * math.expm1(t), False


def exp_quantile_step(mean: float, ratio: float) -> float:
    """Corollary 1.1 / Corollary 2.1: eta = beta_hat * log(1/ratio)."""
    return mean * math.log(1.0 / ratio)


def gamma_shape(s: float) -> float:
    """Closed-form shape estimate of Corollary 1.2."""
    return (3.0 - s + math.sqrt((s - 3.0) ** 2 + 24.0 * s)) / (12.0 * s)


# -- special functions for the exact forms of Corollary 1.2 (plain series; pinned against a library in the tests)

def digamma(x: float) -> float:
    """psi(x) for x > 0: recurrence up to x >= 8, then the asymptotic series."""
    acc = 0.0
    while x < 8.0:
        acc -= 1.0 / x
        x += 1.0
    f = 1.0 / (x * x)
    return acc + math.log(x) - 0.5 / x - f * (1.0 / 12 - f * (1.0 / 120 - f * (1.0 / 252 - f * (1.0 / 240 - f / 132))))


def trigamma(x: float) -> float:
    """psi'(x) for x > 0."""
    acc = 0.0
    while x < 8.0:
        acc += 1.0 / (x * x)
        x += 1.0
    f = 1.0 / (x * x)
    return acc + 1.0 / x + 0.5 * f + (1.0 / x) * f * (1.0 / 6 - f * (1.0 / 30 - f * (1.0 / 42 - f / 30)))


def gamma_shape_mle(s: float) -> float:
    """Maximum-likelihood shape: the root of log(alpha) - psi(alpha) = s (the equation in the proof of
    Corollary 1.2), by Newton's method from the closed-form estimate."""
    alpha = gamma_shape(s)
    for _ in range(100):
        f = math.log(alpha) - digamma(alpha) - s
        step = f / (1.0 / alpha - trigamma(alpha))
        new = alpha - step
        if new <= 0.0:
            new = 0.5 * alpha
        if abs(new - alpha) <= 1e-15 * alpha:
            return new
        alpha = new
    return alpha


def gamma_upper_q(a: float, x: float) -> float:
    """Q(a, x) = 1 - P(a, x), the regularised upper incomplete gamma function: the power series of P for
    x < a + 1, the continued fraction of Q otherwise."""
    if x <= 0.0:
        return 1.0
    log_front = a * math.log(x) - x - math.lgamma(a)
    if x < a + 1.0:
        term = 1.0 / a
        total = term
        n = 0
        while abs(term) > 1e-17 * abs(total) and n < 10000:
            n += 1
            term *= x / (a + n)
            total += term
        return 1.0 - total * math.exp(log_front)
    tiny = 1e-300
    b = x + 1.0 - a
    c = 1.0 / tiny
    d = 1.0 / b
    h = d
    for i in range(1, 10000):
        an = -i * (i - a)
        b += 2.0
        d = an * d + b
        d = tiny if abs(d) < tiny else d
        c = b + an / c
        c = tiny if abs(c) < tiny else c
        d = 1.0 / d
        delta = d * c
        h *= delta
        if abs(delta - 1.0) < 1e-16:
            break
    return h * math.exp(log_front)


def gamma_upper_quantile(a: float, q: float) -> float:
    """x with Q(a, x) = q, i.e. P^{-1}(a, 1 - q): bracketing by doubling, then bisection on log Q refined by
    Newton steps that stay inside the bracket."""
    if q >= 1.0:
        return 0.0
    lo, hi = 0.0, max(1.0, a)
    while gamma_upper_q(a, hi) > q:
        lo, hi = hi, 2.0 * hi
    x = 0.5 * (lo + hi)
    for _ in range(200):
        qx = gamma_upper_q(a, x)
        if qx > q:
            lo = x
        else:
            hi = x
        # Newton on log Q: d/dx log Q = -x^(a-1) e^(-x) / (Gamma(a) Q)
        dens = math.exp((a - 1.0) * math.log(x) - x - math.lgamma(a))
        new = x + (math.log(qx) - math.log(q)) * qx / dens if qx > 0.0 and dens > 0.0 else 0.5 * (lo + hi)
        if not (lo < new < hi):
            new = 0.5 * (lo + hi)
        if abs(new - x) <= 1e-15 * x:
            return new
        x = new
    return x


def gamma_first_stage_exact(a: np.ndarray, ratio: float):
    """Corollary 1.2 without the shortcuts: maximum-likelihood shape and the exact quantile.  Same reading of
    zeros and of constant magnitudes as gamma_first_stage.  Returns (eta, degenerate)."""
    n = a.size
    nz = a[a > 0.0]
    n_nz = nz.size
    mu = float(np.sum(nz)) / n_nz
    s = math.log(mu) - float(np.sum(np.log(nz))) / n_nz
    ratio_nz = min(1.0, ratio * n / n_nz)
    if s <= 1e-12:
        return max(exp_quantile_step(mu, ratio_nz), 0.0), True
    alpha = gamma_shape_mle(s)
    beta = mu / alpha
    return beta * gamma_upper_quantile(alpha, ratio_nz), False


def gamma_first_stage(a: np.ndarray, ratio: float):
    """Corollary 1.2 on the magnitudes ``a`` (fp64).  Returns (eta, degenerate).

    [reading] log|g| of an exact zero is -inf, so the gamma model is fitted to
    the nonzero magnitudes only and the tail probability is rescaled so that it
    still refers to the whole segment."""
    n = a.size
    nz = a[a > 0.0]
    n_nz = nz.size
    mu = float(np.sum(nz)) / n_nz
    s = math.log(mu) - float(np.sum(np.log(nz))) / n_nz
    ratio_nz = min(1.0, ratio * n / n_nz)
    if s <= 1e-12:
        # [reading] constant magnitudes (s = 0 up to rounding; s >= 0 always by
        # Jensen's inequality): fall back to the exponential formula.
        return max(exp_quantile_step(mu, ratio_nz), 0.0), True
    alpha = gamma_shape(s)
    beta = mu / alpha
    eta = -beta * (math.log(ratio_nz) + math.lgamma(alpha))
    if eta <= 0.0:
        # [reading] the closed form goes non-positive when ratio*Gamma(alpha)
        # >= 1; clamp so that every nonzero magnitude exceeds it.
        return 0.0, True
    return eta, False


def thresholds(a: np.ndarray, delta: float, sid: int, M: int, delta1: float,
               policy: Policy = Policy()) -> SegReport:
    """Multi-stage threshold estimation for one segment (Section 2.4).

    ``a`` holds the fp64 magnitudes |acc|.  Stage 1 fits all of them; stage
    m >= 2 fits the shifted exceedances |x| - eta_{m-1} over {|x| > eta_{m-1}}
    (Lemma 2: sample mean and variance of the shifted peaks over threshold) and
    adds the increment to eta_{m-1}."""
    rep = SegReport()
    n = a.size
    M_eff = min(M, stage_cap(delta, delta1))
    rep.M_used = M_eff
    if n == 0:
        rep.eta = [math.inf] * M_eff
        rep.k_stage = [0] * M_eff
        return rep
    if not np.all(np.isfinite(a)):
        # [reading] inputs are assumed finite; otherwise select nothing.
        rep.status |= ST_NONFINITE
        rep.eta = [math.nan] * M_eff
        rep.k_stage = [0] * M_eff
        return rep
    S1 = float(np.sum(a))
    if S1 == 0.0:
        # [reading] an all-zero segment has nothing worth sending.
        rep.status |= ST_ALL_ZERO
        rep.eta = [math.inf] * M_eff
        rep.k_stage = [0] * M_eff
        return rep

    ratios = stage_ratios(delta, M_eff, delta1)

    # ---- stage 1: fit all n magnitudes -----------------------------------
    mu = S1 / n
    if sid == SID_EXP:
        eta = exp_quantile_step(mu, ratios[0])
    elif sid == SID_GPD:
        var = float(np.sum((a - mu) ** 2)) / n      # [reading] population variance
        eta, deg = gpd_quantile_step(mu, var, ratios[0])
        rep.status |= ST_DEGENERATE if deg else 0
    elif sid == SID_GAMMA:
        eta, deg = (gamma_first_stage_exact if policy.gamma_exact else gamma_first_stage)(a, ratios[0])
        rep.status |= ST_DEGENERATE if deg else 0
    else:
        raise ValueError("unknown SID")
    rep.eta.append(eta)

    # ---- stages 2..M: refit on the exceedances ---------------------------
    for m in range(1, M_eff):
        exceed = a[a > eta]                 # strict, as in the stage loop of Algorithm 1
        rep.k_stage.append(int(exceed.size))
        if exceed.size == 0:
            rep.eta.append(eta)             # [reading] nothing left to refit
            continue
        y = exceed - eta
        ybar = float(np.sum(y)) / y.size
        if policy.ratio_from_counts and m == M_eff - 1:
            # the last stage keeps the target count out of what the stage before it left
            ratios[m] = min(1.0, delta * n / exceed.size)
        if sid == SID_EXP:
            inc = exp_quantile_step(ybar, ratios[m])
        else:
            yvar = float(np.sum((y - ybar) ** 2)) / y.size
            inc, deg = gpd_quantile_step(ybar, yvar, ratios[m])
            rep.status |= ST_DEGENERATE if deg else 0
        eta = eta + inc
        rep.eta.append(eta)

    # count for the last threshold is the final selection (non-strict)
    rep.k_stage.append(int(np.count_nonzero(a >= eta)))
    return rep


# ---------------------------------------------------------------------------
# Stage adaptation (Algorithm 1, Adapt_Stages)
# ---------------------------------------------------------------------------

def adapt_stages(M: int, k_avg: float, k: float, eps_H: float, eps_L: float, M_max: int,
                 reversed_direction: bool = False) -> int:
    """Too many selected -> one stage fewer; too few -> one more; clamp.  (reversed_direction: the opposite.)"""
    step = -1 if reversed_direction else 1
    if k_avg > k * (1.0 + eps_H):
        M = M - step
    if k_avg < k * (1.0 - eps_L):
        M = M + step
    return min(max(M, 1), M_max)


def adapt_update(st: SegState, k_hat: int, k: float, params: Params, M_max: int,
                 policy: Policy = Policy()) -> None:
    """[reading] calls are counted from one, every k_hat is added, and the mean
    of exactly Q values is compared at every Q-th call."""
    st.calls += 1
    st.k_sum += int(k_hat)
    if st.calls % params.Q == 0:
        st.M = adapt_stages(st.M, st.k_sum / params.Q, k, params.eps_H, params.eps_L, M_max, policy.adapt_reversed)
        st.k_sum = 0


# ---------------------------------------------------------------------------
# One call of the compressor over a flattened, segmented gradient
# ---------------------------------------------------------------------------

def sidco_compress(grad: np.ndarray, residual: np.ndarray, seg_offsets, delta: float,
                   sid: int, max_stages: int, state: Optional[List[SegState]] = None,
                   params: Params = Params(), policy: Policy = Policy()) -> Result:
    """max_stages > 0: adaptive, M starts at 1 and moves inside [1, max_stages]
    (``state`` is updated in place); max_stages < 0: fixed M = -max_stages."""
    grad = np.asarray(grad, dtype=np.float32)
    residual = np.asarray(residual, dtype=np.float32)
    off = np.asarray(seg_offsets, dtype=np.int64)
    n_segs = off.size - 1
    acc = (grad + residual).astype(np.float32)      # error compensation, fp32
    new_res = acc.copy()
    out_k = np.zeros(n_segs + 1, dtype=np.int32)
    idx_parts, reports = [], []
    adaptive = max_stages > 0
    if adaptive and state is None:
        raise ValueError("adaptive mode needs a state list")
    for s in range(n_segs):
        lo, hi = int(off[s]), int(off[s + 1])
        a = np.abs(acc[lo:hi]).astype(np.float64)
        if adaptive:
            M = min(max(state[s].M, 1), max_stages)
        else:
            M = -max_stages
        rep = thresholds(a, delta, sid, M, params.delta1, policy)
        eta = rep.eta[-1]
        keep = np.nonzero(a >= eta)[0]              # final selection: |x| >= eta_M
        out_k[s] = keep.size
        idx_parts.append(keep + lo)
        reports.append(rep)
        if adaptive:
            adapt_update(state[s], keep.size, delta * (hi - lo), params, max_stages, policy)
    idx = (np.concatenate(idx_parts) if idx_parts else np.zeros(0, np.int64)).astype(np.int32)
    out_k[n_segs] = idx.size
    val = acc[idx]
    new_res[idx] = np.float32(0.0)
    return Result(idx=idx, val=val, out_k=out_k, residual=new_res, acc=acc, report=reports)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """A gradient stored as bf16 enters the error-compensation add widened exactly: bf16 is the upper half
    of an fp32, so the value is the 16 bits followed by 16 zero bits.  (Mixed-precision variant of the
    synthetic-tensor micro-benchmark; the method itself is unchanged.)"""
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def new_state(n_segs: int) -> List[SegState]:
    return [SegState() for _ in range(n_segs)]
