"""Pins for the Top-k and sampled-threshold (DGC-style) oracles of the paper's comparison (Section 1, Fig. 1):
library selection routines, brute force on tiny inputs, invariants, and the known behaviour on a sample."""
import numpy as np
import pytest
import torch

from oracle import reference_points_oracle as R


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


@pytest.mark.parametrize("d,k", [(1, 1), (10, 3), (1000, 1), (1000, 1000), (4097, 41), (50000, 500)])
def test_topk_agrees_with_a_library_topk(d, k):
    r = rng(d + k)
    g = r.standard_normal(d).astype(np.float32)
    res = (0.1 * r.standard_normal(d)).astype(np.float32)
    sel = R.topk_compress(g, res, k)
    acc = g + res
    lib = torch.topk(torch.from_numpy(np.abs(acc)), k)
    # continuous data: no ties, the set is unique
    assert np.array_equal(np.sort(lib.indices.numpy()), sel.idx)
    assert np.array_equal(sel.val, acc[sel.idx]) and np.all(np.diff(sel.idx) > 0)
    assert np.float32(lib.values.min()) == np.uint32(sel.threshold_bits).view(np.float32)
    # what was sent plus what was kept is the accumulated gradient, bit for bit
    back = sel.residual.copy()
    back[sel.idx] = sel.val
    assert np.array_equal(back.view(np.uint32), acc.view(np.uint32)) and not sel.residual[sel.idx].any()


def test_topk_brute_force_with_ties_lowest_index_wins():
    acc = np.array([1.0, -3.0, 3.0, 0.5, -3.0, 2.0, 3.0, -0.5], np.float32)
    zeros = np.zeros_like(acc)
    assert R.topk_compress(acc, zeros, 1).idx.tolist() == [1]
    assert R.topk_compress(acc, zeros, 2).idx.tolist() == [1, 2]
    assert R.topk_compress(acc, zeros, 3).idx.tolist() == [1, 2, 4]
    assert R.topk_compress(acc, zeros, 5).idx.tolist() == [1, 2, 4, 5, 6]
    assert R.topk_compress(acc, zeros, 0).idx.size == 0
    assert R.topk_compress(acc, zeros, 99).idx.tolist() == list(range(8))
    # pure Python definition on random small-integer data (many ties)
    r = rng(4)
    for _ in range(50):
        d = int(r.integers(1, 40))
        a = r.integers(-4, 5, d).astype(np.float32)
        k = int(r.integers(0, d + 1))
        want = sorted(sorted(range(d), key=lambda j: (-abs(float(a[j])), j))[:k])
        assert R.topk_compress(a, np.zeros(d, np.float32), k).idx.tolist() == want


def test_topk_orders_infinities_and_nans_above_finite_values():
    acc = np.array([1.0, np.inf, -2.0, np.nan, 5.0], np.float32)
    assert R.topk_compress(acc, np.zeros(5, np.float32), 2).idx.tolist() == [1, 3]
    assert R.topk_compress(acc, np.zeros(5, np.float32), 3).idx.tolist() == [1, 3, 4]


def test_dgc_threshold_is_the_sample_quantile_and_selection_is_a_plain_threshold():
    d, delta = 200000, 0.01
    r = rng(9)
    g = r.laplace(0.0, 1e-3, d).astype(np.float32)
    res = np.zeros(d, np.float32)
    sample_idx = r.choice(d, d // 100, replace=False)
    sel = R.dgc_compress(g, res, delta, sample_idx)
    thr = np.uint32(sel.threshold_bits).view(np.float32)
    k_s = int(np.ceil(delta * sample_idx.size))
    s = np.abs(g[sample_idx])
    assert thr == np.partition(s, s.size - k_s)[s.size - k_s]          # library order statistic
    assert np.count_nonzero(s >= thr) == k_s
    assert np.array_equal(sel.idx, np.nonzero(np.abs(g) >= thr)[0])
    # the achieved count follows the sample: unbiased up to the sampling error of an order statistic
    k = delta * d
    assert abs(sel.idx.size - k) < 6 * k / np.sqrt(k_s)
    # Laplace data: the threshold estimates b * ln(1 / delta)
    assert thr == pytest.approx(1e-3 * np.log(1 / delta), rel=0.25)


def test_dgc_full_sample_is_exact_topk_when_there_are_no_ties():
    d, delta = 5000, 0.02
    r = rng(10)
    g = r.standard_normal(d).astype(np.float32)
    res = (0.3 * r.standard_normal(d)).astype(np.float32)
    a = R.dgc_compress(g, res, delta, np.arange(d))
    b = R.topk_compress(g, res, int(np.ceil(delta * d)))
    assert np.array_equal(a.idx, b.idx) and a.threshold_bits == b.threshold_bits


def test_dgc_degenerate_samples():
    g = np.array([0.5, -2.0, 1.0], np.float32)
    z = np.zeros(3, np.float32)
    assert R.dgc_compress(g, z, 0.5, np.zeros(0, np.int64)).idx.size == 0
    assert R.dgc_compress(g, z, 1e-9, np.array([2])).idx.tolist() == [1, 2]        # k_s is at least one
    assert R.dgc_compress(g, z, 1.0, np.array([0, 1, 2])).idx.tolist() == [0, 1, 2]
