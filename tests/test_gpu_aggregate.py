"""sidco_aggregate (dense mean of N workers' sparse lists, the collective step of the paper's sparsified
synchronous SGD) against the aggregation oracle: bit-exact, through the C ABI."""
import numpy as np
import pytest

from oracle import aggregate_oracle as A
from oracle import sidco_oracle as O
from paper_2101_10761_b200 import workloads as W

pytestmark = pytest.mark.gpu


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def pack(idx_lists, val_lists, stride=None):
    n = len(idx_lists)
    counts = np.array([len(i) for i in idx_lists], np.int32)
    if stride is None:
        stride = max(8, (int(counts.max()) + 7) // 8 * 8)
    idx_all = np.full(n * stride, 0x7fffffff, np.int32)          # padding that must never be read as an index
    val_all = np.full(n * stride, np.nan, np.float32)
    for w in range(n):
        idx_all[w * stride:w * stride + counts[w]] = idx_lists[w]
        val_all[w * stride:w * stride + counts[w]] = val_lists[w]
    return idx_all, val_all, counts, stride


def run_gpu(idx_lists, val_lists, d, shift=0, stride=None):
    import torch
    from paper_2101_10761_b200 import binding as B
    dev = "cuda:0"
    idx_all, val_all, counts, stride = pack(idx_lists, val_lists, stride)
    store = torch.full((d + 16,), 7.0, dtype=torch.float32, device=dev)         # stale contents must be overwritten
    out = store[shift:shift + d]
    status = torch.full((1,), -1, dtype=torch.int32, device=dev)
    B.sidco_aggregate(torch.from_numpy(idx_all).to(dev), torch.from_numpy(val_all).to(dev),
                      torch.from_numpy(counts).to(dev), len(idx_lists), stride, d, out, status)
    torch.cuda.synchronize()
    assert float(store[shift + d]) == 7.0 and (shift == 0 or float(store[shift - 1]) == 7.0), "wrote outside out_dense"
    return out.cpu().numpy(), int(status.item())


def random_lists(seed, d, n_workers, density, overlap=0.5):
    r = rng(seed)
    shared = r.random(d) < density * overlap
    idx, val = [], []
    for _ in range(n_workers):
        keep = np.nonzero(shared | (r.random(d) < density * (1 - overlap)))[0].astype(np.int32)
        idx.append(keep)
        val.append(r.standard_normal(keep.size).astype(np.float32) * np.float32(1e-3))
    return idx, val


@pytest.mark.parametrize("d,n_workers,density,shift", [
    (1, 1, 1.0, 0), (7, 3, 0.5, 0), (4095, 2, 0.01, 0), (4096, 8, 0.001, 0), (4097, 8, 0.2, 1),
    (100003, 5, 0.01, 3), (1 << 20, 8, 0.001, 0), (3000017, 16, 0.002, 0), (600001, 64, 0.0005, 0)])
def test_matches_the_oracle_bit_for_bit(d, n_workers, density, shift):
    idx, val = random_lists(d % 1000 + n_workers, d, n_workers, density)
    want = A.aggregate(idx, val, d)
    got, status = run_gpu(idx, val, d, shift)
    assert status == 0
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_dense_lists_take_the_global_memory_path():
    # every worker sends a third of all positions: far more entries per CTA range than shared memory holds
    d, n_workers = 2_000_003, 6
    idx, val = random_lists(77, d, n_workers, 0.33, overlap=0.8)
    want = A.aggregate(idx, val, d)
    got, status = run_gpu(idx, val, d)
    assert status == 0
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_empty_lists_and_signed_zeros():
    d = 50000
    idx = [np.zeros(0, np.int32), np.array([5, 49999], np.int32), np.array([5], np.int32)]
    val = [np.zeros(0, np.float32), np.array([-0.0, 2.5], np.float32), np.array([-0.0], np.float32)]
    want = A.aggregate(idx, val, d)
    got, status = run_gpu(idx, val, d, stride=24)
    assert status == 0 and np.array_equal(got.view(np.uint32), want.view(np.uint32))
    got, status = run_gpu([np.zeros(0, np.int32)] * 4, [np.zeros(0, np.float32)] * 4, d)
    assert status == 0 and not got.any() and not np.signbit(got).any()


def test_output_of_eight_compress_calls_on_the_resnet50_shaped_workload():
    """N = 8 workers, each compressing its own draw of the d = 25.6 M workload (delta = 1e-3) on the GPU; the
    gathered lists are aggregated on the GPU and compared with the oracle's aggregate of the same lists."""
    import torch
    from paper_2101_10761_b200 import binding as B
    dev = "cuda:0"
    wl = W.config(4)
    d, S, off = wl.d, wl.n_segs, wl.seg_offsets
    res = torch.zeros(d, dtype=torch.float32, device=dev)
    out_idx = torch.empty(d, dtype=torch.int32, device=dev)
    out_val = torch.empty(d, dtype=torch.float32, device=dev)
    out_k = torch.zeros(S + 1, dtype=torch.int32, device=dev)
    idx, val = [], []
    try:
        for w in range(8):
            res.zero_()
            B.sidco_compress(torch.from_numpy(wl.draw(40 + w)).to(dev), res, off, float(np.float32(1e-3)), 0, -1,
                             out_idx, out_val, out_k)
            torch.cuda.synchronize()
            k = int(out_k[S])
            idx.append(out_idx[:k].cpu().numpy())
            val.append(out_val[:k].cpu().numpy())
    finally:
        B.sidco_release(res)
    del res, out_idx, out_val
    want = A.aggregate(idx, val, d)
    got, status = run_gpu(idx, val, d)
    assert status == 0
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert np.count_nonzero(got) > 0


def test_bad_counts_and_unordered_lists_are_reported_not_trusted():
    import torch
    from paper_2101_10761_b200 import binding as B
    dev = "cuda:0"
    d, stride = 30000, 16
    idx_all = np.zeros(2 * stride, np.int32)
    val_all = np.ones(2 * stride, np.float32)
    idx_all[:4] = [3, 100, 200, 29999]
    idx_all[stride:stride + 3] = [20000, 7, 25000]          # not ascending
    counts = np.array([4, 99], np.int32)                     # second count exceeds the stride
    out = torch.empty(d, dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.sidco_aggregate(torch.from_numpy(idx_all).to(dev), torch.from_numpy(val_all).to(dev),
                      torch.from_numpy(counts).to(dev), 2, stride, d, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) & B.AGG_ST_COUNT
    got = out.cpu().numpy()
    assert got[3] == 0.5 and got[29999] == 0.5 and np.isfinite(got).all()
    with pytest.raises(B.SidcoError):
        B.sidco_aggregate(out, out, out, 0, stride, d, out, None)
    with pytest.raises(B.SidcoError):
        B.sidco_aggregate(out, out, out, 65, stride, d, out, None)
    with pytest.raises(B.SidcoError):
        B.sidco_aggregate(None, out, out, 2, stride, d, out, None)
