"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI
binding and compare with the oracle under the stated tolerances."""
import math

import numpy as np

from oracle import sidco_oracle as O

ETA_RTOL = 1e-6       # threshold: relative error vs the oracle
BAND_RTOL = 1e-6      # indices may differ only where | |x| - eta | <= BAND_RTOL * eta


def f32(x: float) -> float:
    """The float the C ABI receives for a Python delta."""
    return float(np.float32(x))


class GpuRun:
    """One residual buffer on the device with its output buffers; call step() repeatedly."""

    def __init__(self, offsets, residual0=None, base_shift=0):
        import torch
        from paper_2101_10761_b200 import binding as B
        self.torch, self.B = torch, B
        self.off = np.asarray(offsets, dtype=np.int64)
        self.S = self.off.size - 1
        self.d = int(self.off[-1])
        dev = "cuda:0"
        cap = self.d + 8 + base_shift
        # base_shift > 0 gives pointers that are not 32-byte aligned (scalar path)
        self._res_store = torch.zeros(cap, dtype=torch.float32, device=dev)
        self._grad_store = torch.zeros(cap, dtype=torch.float32, device=dev)
        self.res = self._res_store[base_shift:base_shift + self.d]
        self.grad = self._grad_store[base_shift:base_shift + self.d]
        self.out_idx = torch.full((self.d + 8,), -7, dtype=torch.int32, device=dev)
        self.out_val = torch.zeros(self.d + 8, dtype=torch.float32, device=dev)
        self.out_k = torch.full((self.S + 1,), -7, dtype=torch.int32, device=dev)
        if residual0 is not None:
            self.res.copy_(torch.from_numpy(np.asarray(residual0, dtype=np.float32)))

    def step(self, grad, delta, sid, max_stages):
        torch, B = self.torch, self.B
        self.grad.copy_(torch.from_numpy(np.asarray(grad, dtype=np.float32)))
        ptr_g = self.grad.data_ptr() if self.d else self._grad_store.data_ptr()
        ptr_r = self.res.data_ptr() if self.d else self._res_store.data_ptr()
        self.key = ptr_r
        B.sidco_compress(ptr_g, ptr_r, self.off, delta, sid, max_stages,
                         self.out_idx, self.out_val, self.out_k)
        torch.cuda.synchronize()
        out_k = self.out_k.cpu().numpy()
        k = int(out_k[-1])
        return dict(idx=self.out_idx[:k].cpu().numpy(), val=self.out_val[:k].cpu().numpy(), out_k=out_k,
                    residual=self.res.cpu().numpy(), debug=B.sidco_get_debug(ptr_r, self.S))

    def close(self):
        self.B.sidco_release(self.key)


def eta_close(a: float, b: float) -> bool:
    if math.isnan(a) or math.isnan(b):
        return math.isnan(a) and math.isnan(b)
    if math.isinf(a) or math.isinf(b):
        return a == b
    return abs(a - b) <= ETA_RTOL * abs(b)


def check_parity(gpu, ora: O.Result, offsets, state=None, check_status=True):
    """Element-by-element comparison of one call.  Returns the number of tolerated band elements."""
    off = np.asarray(offsets, dtype=np.int64)
    S = off.size - 1
    acc = ora.acc
    band_total = 0
    # thresholds, stage counts, status
    for s in range(S):
        rep, dbg = ora.report[s], gpu["debug"][s]
        assert dbg.M_used == rep.M_used, f"seg {s}: M_used {dbg.M_used} vs {rep.M_used}"
        for m in range(rep.M_used):
            assert eta_close(dbg.eta[m], rep.eta[m]), f"seg {s} stage {m}: eta {dbg.eta[m]!r} vs {rep.eta[m]!r}"
        if check_status:
            assert dbg.status == rep.status, f"seg {s}: status {dbg.status} vs {rep.status}"
        if state is not None:
            assert dbg.M_next == state[s].M and dbg.calls == state[s].calls and dbg.k_sum == state[s].k_sum, \
                f"seg {s}: adaptation state ({dbg.M_next},{dbg.calls},{dbg.k_sum}) vs " \
                f"({state[s].M},{state[s].calls},{state[s].k_sum})"
    # indices: identical up to elements inside the tolerance band around eta
    g_idx, o_idx = gpu["idx"].astype(np.int64), ora.idx.astype(np.int64)
    assert np.all(np.diff(g_idx) > 0), "GPU indices not strictly ascending"
    assert int(gpu["out_k"][-1]) == g_idx.size
    diff = np.setxor1d(g_idx, o_idx)
    if diff.size:
        seg_of = np.searchsorted(off, diff, side="right") - 1
        for j, s in zip(diff, seg_of):
            eta = ora.report[s].eta[-1]
            assert abs(abs(float(acc[j])) - eta) <= BAND_RTOL * eta, \
                f"index {j} (seg {s}) differs outside the band: |x|={abs(float(acc[j]))!r} eta={eta!r}"
            # the band is there for thresholds that differ in their last bits; with the same threshold on both
            # sides the comparison |x| >= eta has one answer
            assert gpu["debug"][s].eta[ora.report[s].M_used - 1] != eta, \
                f"index {j} (seg {s}): same threshold {eta!r} on both sides but different selections"
        band_total = diff.size
    # per-segment counts agree with the GPU's own index list
    counts = np.bincount(np.searchsorted(off[1:], g_idx, side="right"), minlength=S)[:S] if g_idx.size else np.zeros(S, int)
    assert np.array_equal(gpu["out_k"][:S], counts.astype(np.int32)), "out_k does not match the index list"
    if not diff.size:
        assert np.array_equal(gpu["out_k"], ora.out_k)
        for s in range(S):
            rep, dbg = ora.report[s], gpu["debug"][s]
            assert list(dbg.k_stage[:rep.M_used]) == rep.k_stage, f"seg {s}: stage counts {list(dbg.k_stage[:rep.M_used])} vs {rep.k_stage}"
    # values and residual: bit exact (outside the band elements)
    assert np.array_equal(gpu["val"].view(np.uint32), acc[g_idx].view(np.uint32)), "out_val != acc[out_idx]"
    exp_res = acc.copy()
    exp_res[g_idx] = np.float32(0.0)
    assert np.array_equal(gpu["residual"].view(np.uint32), exp_res.view(np.uint32)), "residual mismatch"
    if not diff.size:
        assert np.array_equal(gpu["residual"].view(np.uint32), ora.residual.view(np.uint32))
    return band_total
