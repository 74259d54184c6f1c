"""CPU oracle for the aggregation step that follows the sparsifier (test infrastructure only).

In the sparsified distributed synchronous SGD of the paper's appendix (the algorithm box "Sparsified
Distributed Synchronous SGD"), every one of the N workers sparsifies its own gradient and the collective
step forms

    G = (1/N) * sum_{n=1..N} Sparsify(g_n, delta)

i.e. the dense mean of the N sparse vectors.  Worker n's sparse vector arrives as an ascending list of
(index, value) pairs; positions that no worker sent are zero.

This is the definition written out: an fp64 accumulator per position, the workers added in the order
n = 1..N, one division by N, one rounding to fp32.  It is NOT part of the product and shares no code with
the CUDA path; only tests, the smoke check and the benchmark's CPU leg may import it.

Pins (tests/test_aggregate_oracle_pins.py): exact rational arithmetic on small inputs, the single-worker
and disjoint-support special cases, agreement with the mean of dense vectors when every list is complete,
and conservation together with the compress oracle (what a worker sent plus what it kept is its
accumulated gradient).
"""
from __future__ import annotations

from typing import Sequence

import numpy as np


def aggregate(idx_lists: Sequence[np.ndarray], val_lists: Sequence[np.ndarray], d: int) -> np.ndarray:
    """Dense mean of N sparse vectors of length d.  idx_lists[n] is strictly ascending (no position twice
    within one worker), val_lists[n] holds the fp32 values at those positions.  Returns fp32[d]."""
    n_workers = len(idx_lists)
    if n_workers < 1 or len(val_lists) != n_workers:
        raise ValueError("need one index list and one value list per worker")
    acc = np.zeros(d, dtype=np.float64)
    for idx, val in zip(idx_lists, val_lists):
        idx = np.asarray(idx, dtype=np.int64)
        val = np.asarray(val, dtype=np.float32)
        if idx.size != val.size:
            raise ValueError("index and value lists differ in length")
        if idx.size and (idx[0] < 0 or idx[-1] >= d or np.any(np.diff(idx) <= 0)):
            raise ValueError("indices must be strictly ascending and inside [0, d)")
        acc[idx] += val.astype(np.float64)        # distinct positions: one addition each, worker order
    return (acc / float(n_workers)).astype(np.float32)
