"""CPU oracles for the two compressors the paper measures its own against (test infrastructure only).

Section 1 and Fig. 1 of the paper compare threshold estimation with (i) exact Top-k selection and (ii) the
sampled-threshold scheme of Deep Gradient Compression (DGC): a small random sample of the gradient is taken,
Top-k is run on the sample only, and the k-th largest sampled magnitude is used as the threshold for the
whole vector.  Both are stated here in the plainest form, with the same error-compensation wrapper as the
SIDCo path (acc = g + residual in fp32; survivors leave the residual), so that the three can be timed and
their achieved ratios k_hat / k compared on the same inputs.  Whole-vector selection, as in the paper's
micro-benchmark.

Not part of the product; shares no code with the CUDA path.

Order of equal magnitudes (several answers would be "a" Top-k): magnitudes are compared as the bit patterns
of |acc| (which orders finite values, puts infinities above them and NaNs above those), and among equal
magnitudes the lower index wins.  That makes the selected set unique.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class Selection:
    idx: np.ndarray          # int32, ascending
    val: np.ndarray          # float32, acc at idx
    residual: np.ndarray     # float32[d], acc with the selected entries set to +0
    acc: np.ndarray          # float32[d]
    threshold_bits: int      # bit pattern of the smallest selected magnitude (0 if nothing was selected)


def _keys(acc: np.ndarray) -> np.ndarray:
    return acc.view(np.uint32) & np.uint32(0x7FFFFFFF)


def _finish(acc: np.ndarray, idx: np.ndarray, thr_bits: int) -> Selection:
    idx = np.sort(idx).astype(np.int32)
    res = acc.copy()
    res[idx] = np.float32(0.0)
    return Selection(idx=idx, val=acc[idx], residual=res, acc=acc, threshold_bits=int(thr_bits))


def topk_compress(grad: np.ndarray, residual: np.ndarray, k: int) -> Selection:
    """Exact Top-k of |g + residual| by a full sort (definition, not an algorithm)."""
    acc = (np.asarray(grad, np.float32) + np.asarray(residual, np.float32)).astype(np.float32)
    d = acc.size
    k = max(0, min(int(k), d))
    if k == 0:
        return _finish(acc, np.zeros(0, np.int64), 0)
    keys = _keys(acc).astype(np.int64)
    # descending magnitude, ascending index among equals
    order = np.lexsort((np.arange(d), -keys))
    chosen = order[:k]
    return _finish(acc, chosen, int(keys[chosen[-1]]))


def dgc_compress(grad: np.ndarray, residual: np.ndarray, delta: float, sample_idx: np.ndarray) -> Selection:
    """Sampled threshold: Top-k on the sample only (k_s = ceil(delta * n_s), at least 1), then every element
    of the whole vector whose magnitude reaches the k_s-th largest sampled magnitude."""
    acc = (np.asarray(grad, np.float32) + np.asarray(residual, np.float32)).astype(np.float32)
    keys = _keys(acc)
    sample = keys[np.asarray(sample_idx, dtype=np.int64)]
    n_s = sample.size
    if n_s == 0:
        return _finish(acc, np.zeros(0, np.int64), 0)
    k_s = max(1, min(n_s, int(np.ceil(float(delta) * n_s))))
    thr = np.sort(sample)[n_s - k_s]                  # k_s-th largest sampled magnitude
    return _finish(acc, np.nonzero(keys >= thr)[0], int(thr))
