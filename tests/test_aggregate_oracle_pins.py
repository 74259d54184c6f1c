"""Pins for the aggregation oracle (dense mean of N workers' sparse lists, the collective step of the
paper's sparsified synchronous SGD): exact rational arithmetic, special cases with a textbook answer,
agreement with a dense mean, and conservation together with the compress oracle."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import aggregate_oracle as A
from oracle import sidco_oracle as O


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def random_lists(seed, d, n_workers, density):
    r = rng(seed)
    idx, val = [], []
    for _ in range(n_workers):
        keep = np.nonzero(r.random(d) < density)[0]
        idx.append(keep.astype(np.int32))
        # multiples of 2^-10 below 2^6: every partial sum of up to 64 of them is exact in fp64 and in fp32
        val.append((r.integers(-2 ** 12, 2 ** 12, keep.size) / 1024.0).astype(np.float32))
    return idx, val


@pytest.mark.parametrize("n_workers", [1, 2, 3, 8])
def test_exact_rational_arithmetic_on_small_inputs(n_workers):
    d = 97
    idx, val = random_lists(10 + n_workers, d, n_workers, 0.3)
    got = A.aggregate(idx, val, d)
    want = [Fraction(0)] * d
    for i_w, v_w in zip(idx, val):
        for i, v in zip(i_w.tolist(), v_w.tolist()):
            want[i] += Fraction(v)
    for j in range(d):
        exact = want[j] / n_workers
        # the sum is exact by construction, so the only roundings are the division and the cast
        assert got[j] == np.float32(float(exact)), (j, got[j], float(exact))
    assert got.dtype == np.float32 and got.shape == (d,)


def test_single_worker_is_a_scatter():
    d = 1000
    idx, val = random_lists(3, d, 1, 0.05)
    got = A.aggregate(idx, val, d)
    dense = np.zeros(d, np.float32)
    dense[idx[0]] = val[0]
    assert np.array_equal(got, dense)


def test_disjoint_supports_divide_each_value_by_n():
    d, n_workers = 4096, 4
    r = rng(5)
    perm = r.permutation(d)[:400]
    parts = np.array_split(np.sort(perm[:200]), 1) + [np.sort(perm[200 + 50 * w:250 + 50 * w]) for w in range(3)]
    vals = [r.standard_normal(p.size).astype(np.float32) for p in parts]
    got = A.aggregate(parts, vals, d)
    for p, v in zip(parts, vals):
        assert np.array_equal(got[p], (v / np.float32(n_workers)))      # a division by 4 is exact in fp32
    untouched = np.setdiff1d(np.arange(d), np.concatenate(parts))
    assert np.all(got[untouched] == 0.0) and not np.any(np.signbit(got[untouched]))


def test_complete_lists_give_the_dense_mean():
    d, n_workers = 513, 5
    r = rng(8)
    dense = r.standard_normal((n_workers, d)).astype(np.float32)
    idx = [np.arange(d, dtype=np.int32)] * n_workers
    got = A.aggregate(idx, list(dense), d)
    want = dense.astype(np.float64).mean(axis=0)
    assert np.allclose(got, want, rtol=0, atol=1e-7 * np.abs(dense).sum(axis=0).max())
    # and against a correctly rounded sum (math.fsum) to within one fp32 rounding of the fp64 result
    import math
    for j in range(0, d, 37):
        exact = math.fsum(float(x) for x in dense[:, j]) / n_workers
        assert abs(float(got[j]) - exact) <= 2.0 ** -24 * abs(exact) + 1e-16 * np.abs(dense[:, j]).sum()


def test_worker_order_is_the_summation_order():
    # three values whose fp64 sum depends on the order: (1 + 2^-60) - 1 versus 1 - 1 + 2^-60
    d = 4
    one, tiny = np.float32(1.0), np.float32(2.0 ** -60)
    a = A.aggregate([np.array([2]), np.array([2]), np.array([2])],
                    [np.array([one]), np.array([tiny]), np.array([-one])], d)
    b = A.aggregate([np.array([2]), np.array([2]), np.array([2])],
                    [np.array([one]), np.array([-one]), np.array([tiny])], d)
    assert a[2] == 0.0 and b[2] == np.float32(2.0 ** -60 / 3.0)


def test_rejects_malformed_lists():
    with pytest.raises(ValueError):
        A.aggregate([np.array([3, 3])], [np.array([1.0, 2.0], np.float32)], 10)
    with pytest.raises(ValueError):
        A.aggregate([np.array([1, 12])], [np.array([1.0, 2.0], np.float32)], 10)
    with pytest.raises(ValueError):
        A.aggregate([np.array([1, 2])], [np.array([1.0], np.float32)], 10)


def test_conservation_with_the_compress_oracle():
    """What every worker sent plus what it kept in its error-compensation memory is its accumulated
    gradient, so N * G + sum of residuals = sum of (g_n + old residual_n)."""
    d, n_workers = 6000, 4
    off = [0, 2500, 2501, 6000]
    r = rng(21)
    idx, val, kept, accs = [], [], [], []
    for w in range(n_workers):
        g = r.laplace(0.0, 1e-3, d).astype(np.float32)
        res0 = r.laplace(0.0, 2e-4, d).astype(np.float32)
        out = O.sidco_compress(g, res0, off, 0.05, O.SID_EXP, -2)
        idx.append(out.idx)
        val.append(out.val)
        kept.append(out.residual.astype(np.float64))
        accs.append(out.acc.astype(np.float64))
    G = A.aggregate(idx, val, d).astype(np.float64)
    lhs = n_workers * G + np.sum(kept, axis=0)
    rhs = np.sum(accs, axis=0)
    assert np.allclose(lhs, rhs, rtol=0, atol=4 * 2.0 ** -24 * np.abs(rhs).max() * n_workers)
