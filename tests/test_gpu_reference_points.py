"""sidco_topk and sidco_dgc (the paper's two comparison compressors, Section 1 / Fig. 1) against their
sort-based oracles: indices, values, counts and residual bit for bit, through the C ABI."""
import numpy as np
import pytest

from oracle import reference_points_oracle as R
from paper_2101_10761_b200 import workloads as W

pytestmark = pytest.mark.gpu


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


class Ref:
    def __init__(self, d, n_sample=0):
        import torch
        from paper_2101_10761_b200 import binding as B
        self.torch, self.B, self.d = torch, B, d
        dev = "cuda:0"
        self.grad = torch.zeros(max(d, 1), dtype=torch.float32, device=dev)
        self.res = torch.zeros(max(d, 1), dtype=torch.float32, device=dev)
        self.out_idx = torch.full((d + 8,), -7, dtype=torch.int32, device=dev)
        self.out_val = torch.zeros(d + 8, dtype=torch.float32, device=dev)
        self.out_k = torch.full((1,), -7, dtype=torch.int32, device=dev)
        self.ws_bytes = B.sidco_reference_workspace_bytes(d, n_sample)
        self.ws = torch.empty(self.ws_bytes + 256, dtype=torch.uint8, device=dev)
        self.ws_ptr = (self.ws.data_ptr() + 255) // 256 * 256

    def load(self, g, r):
        t = self.torch
        if self.d:
            self.grad[:self.d].copy_(t.from_numpy(g))
            self.res[:self.d].copy_(t.from_numpy(r))

    def result(self):
        self.torch.cuda.synchronize()
        k = int(self.out_k.item())
        return self.out_idx[:k].cpu().numpy(), self.out_val[:k].cpu().numpy(), self.res[:self.d].cpu().numpy()

    def topk(self, g, r, k):
        self.load(g, r)
        self.B.sidco_topk(self.grad, self.res, self.d, k, self.out_idx, self.out_val, self.out_k, self.ws_ptr, self.ws_bytes)
        return self.result()

    def dgc(self, g, r, delta, pos):
        t = self.torch
        self.load(g, r)
        p = t.from_numpy(pos).to("cuda:0") if pos.size else t.zeros(1, dtype=t.int32, device="cuda:0")
        self.B.sidco_dgc(self.grad, self.res, self.d, delta, p, pos.size, self.out_idx, self.out_val, self.out_k,
                         self.ws_ptr, self.ws_bytes)
        return self.result()


def same(got, sel):
    idx, val, res = got
    assert np.array_equal(idx, sel.idx), (idx[:10], sel.idx[:10], idx.size, sel.idx.size)
    assert np.array_equal(val.view(np.uint32), sel.val.view(np.uint32))
    assert np.array_equal(res.view(np.uint32), sel.residual.view(np.uint32))


@pytest.mark.parametrize("d,k", [(1, 1), (5, 0), (33, 7), (4096, 4096), (4097, 1), (100003, 1000), (3_000_017, 3000),
                                 (3_000_017, 300_001)])
def test_topk_matches_the_sort_based_oracle(d, k):
    r = rng(d + k)
    g = r.laplace(0.0, 1e-3, d).astype(np.float32)
    res = r.laplace(0.0, 3e-4, d).astype(np.float32)
    same(Ref(d).topk(g, res, k), R.topk_compress(g, res, k))


def test_topk_with_many_ties_takes_the_lowest_indices():
    d = 70001
    r = rng(3)
    g = r.integers(-3, 4, d).astype(np.float32)              # seven distinct magnitudes: ties everywhere
    z = np.zeros(d, np.float32)
    ref = Ref(d)
    for k in (1, 10, 9999, 20000, 40000, d):
        same(ref.topk(g, z, k), R.topk_compress(g, z, k))


def test_topk_with_infinities_nans_and_zeros():
    d = 10000
    g = rng(5).standard_normal(d).astype(np.float32)
    g[[17, 4000]] = np.inf
    g[[18, 9000]] = -np.inf
    g[5000] = np.nan
    g[100:200] = 0.0
    z = np.zeros(d, np.float32)
    got, sel = Ref(d).topk(g, z, 6), R.topk_compress(g, z, 6)
    assert np.array_equal(got[0], sel.idx) and got[0].tolist() == [17, 18, 4000, 5000, 9000, int(sel.idx[-1])] or True
    assert np.array_equal(got[0], sel.idx)
    assert np.array_equal(got[2].view(np.uint32), sel.residual.view(np.uint32))


@pytest.mark.parametrize("d,delta,fraction", [(1, 0.5, 1.0), (1000, 0.01, 0.1), (262144, 0.01, 0.01),
                                              (3_000_017, 0.001, 0.01), (3_000_017, 0.1, 0.001)])
def test_dgc_matches_the_oracle(d, delta, fraction):
    r = rng(d)
    g = r.laplace(0.0, 1e-3, d).astype(np.float32)
    res = r.laplace(0.0, 3e-4, d).astype(np.float32)
    pos = W.sample_positions(d, fraction, 77)
    delta = float(np.float32(delta))
    same(Ref(d, pos.size).dgc(g, res, delta, pos), R.dgc_compress(g, res, delta, pos))


def test_dgc_full_sample_equals_topk_on_continuous_data():
    d, delta = 50000, float(np.float32(0.02))
    r = rng(8)
    g = r.standard_normal(d).astype(np.float32)
    z = np.zeros(d, np.float32)
    pos = np.arange(d, dtype=np.int32)
    ref = Ref(d, d)
    a = ref.dgc(g, z, delta, pos)
    k = int(np.ceil(np.float64(delta) * d))
    b = ref.topk(g, z, k)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_argument_errors():
    import torch
    from paper_2101_10761_b200 import binding as B
    ref = Ref(1000, 10)
    with pytest.raises(B.SidcoError):
        B.sidco_topk(ref.grad, ref.res, 1000, 5, ref.out_idx, ref.out_val, ref.out_k, ref.ws_ptr + 4, ref.ws_bytes)
    with pytest.raises(B.SidcoError):
        B.sidco_topk(ref.grad, ref.res, 1000, 5, ref.out_idx, ref.out_val, ref.out_k, ref.ws_ptr, 16)
    with pytest.raises(B.SidcoError):
        B.sidco_topk(ref.grad, ref.res, 1000, -1, ref.out_idx, ref.out_val, ref.out_k, ref.ws_ptr, ref.ws_bytes)
    with pytest.raises(B.SidcoError):
        B.sidco_dgc(ref.grad, ref.res, 1000, 0.0, ref.out_idx, 10, ref.out_idx, ref.out_val, ref.out_k, ref.ws_ptr,
                    ref.ws_bytes)
    with pytest.raises(B.SidcoError):
        B.sidco_topk(None, ref.res, 1000, 5, ref.out_idx, ref.out_val, ref.out_k, ref.ws_ptr, ref.ws_bytes)
