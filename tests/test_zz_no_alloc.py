"""sidco_compress_static: the entry point for callers that must not allocate device memory (stream
capture in progress, all device memory owned by a framework's pool, loops that cannot afford the
implicit synchronisation of cudaMalloc).  Its scratch is a fixed array inside the library, so the
test is simply: through the C ABI, it must produce what sidco_compress produces, on two calls in a
row (the second call reuses the scratch and the adaptation state the first one left behind).

Collected last on purpose: a failure here cannot hide failures of the other GPU tests under -x."""
import numpy as np
import pytest

from paper_2101_10761_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _buffers(d, n_segs, dev):
    import torch
    return (torch.zeros(d, dtype=torch.float32, device=dev), torch.zeros(d, dtype=torch.float32, device=dev),
            torch.full((d,), -3, dtype=torch.int32, device=dev), torch.zeros(d, dtype=torch.float32, device=dev),
            torch.full((n_segs + 1,), -3, dtype=torch.int32, device=dev))


@pytest.mark.parametrize("sid,max_stages", [(0, 3), (1, -1), (2, -3)])
def test_static_entry_matches_allocating_entry_on_two_calls(sid, max_stages):
    import torch
    from paper_2101_10761_b200 import binding as B
    dev = "cuda:0"
    wl = W.config(2)                       # 269,722 elements in 20 segments, within the static limits
    off, d, S = wl.seg_offsets, wl.d, wl.n_segs
    assert d <= B.STATIC_MAX_ELEMS and S <= B.STATIC_MAX_SEGS
    delta = float(np.float32(0.01))
    g_a, r_a, i_a, v_a, k_a = _buffers(d, S, dev)       # allocating entry point
    g_s, r_s, i_s, v_s, k_s = _buffers(d, S, dev)       # allocation-free entry point
    try:
        for call in range(2):
            g = torch.from_numpy(wl.draw(call)).to(dev)
            g_a.copy_(g)
            g_s.copy_(g)
            B.sidco_compress(g_a, r_a, off, delta, sid, max_stages, i_a, v_a, k_a)
            B.sidco_compress_static(g_s, r_s, off, delta, sid, max_stages, i_s, v_s, k_s)
            torch.cuda.synchronize()
            k = int(k_a[S])
            assert k > 0
            # same kernel, same arithmetic: thresholds are identical, so the comparison is exact,
            # which is inside the tolerances the parity tests allow
            assert torch.equal(k_s, k_a)
            assert torch.equal(i_s[:k], i_a[:k])
            assert torch.equal(v_s[:k].view(torch.int32), v_a[:k].view(torch.int32))
            assert torch.equal(r_s.view(torch.int32), r_a.view(torch.int32))
    finally:
        B.sidco_release(r_a)


def test_static_entry_rejects_sizes_beyond_its_limit():
    import torch
    from paper_2101_10761_b200 import binding as B
    dev = "cuda:0"
    n = B.STATIC_MAX_ELEMS + 4
    g, r, i, v, k = _buffers(n, 1, dev)
    with pytest.raises(B.SidcoError) as err:
        B.sidco_compress_static(g, r, [0, n], 0.01, 0, 1, i, v, k)
    assert err.value.code == -10 and "limit" in str(err.value)
    too_many = list(range(0, B.STATIC_MAX_SEGS + 2))
    g, r, i, v, k = _buffers(len(too_many), len(too_many) - 1, dev)
    with pytest.raises(B.SidcoError) as err:
        B.sidco_compress_static(g, r, too_many, 0.01, 0, 1, i, v, k)
    assert err.value.code == -10
