"""sidco_compress_static: the entry point for callers that must not allocate device memory (stream
capture in progress, all device memory owned by a framework's pool, loops that cannot afford the
implicit synchronisation of cudaMalloc).  Its scratch is a fixed array inside the library, so the
tests are: through the C ABI, it must produce what sidco_compress produces (and what the oracle
computes) on consecutive calls, the second of which reuses the scratch and the adaptation state the
first one left behind; the one piece of logic it has of its own - re-keying the shared array when
another residual or another segment table comes along - must leave nothing of the previous pair
behind; and the calls it has to refuse must enqueue nothing.

Collected last on purpose: a failure here cannot hide failures of the other GPU tests under -x."""
import numpy as np
import pytest

from oracle import sidco_oracle as O
from paper_2101_10761_b200 import workloads as W
from parity_util import check_parity, f32

pytestmark = pytest.mark.gpu


def _buffers(d, n_segs, dev, shift=0):
    import torch
    store = [torch.zeros(d + 16, dtype=torch.float32, device=dev) for _ in range(2)]
    return (store[0][shift:shift + d], store[1][shift:shift + d],
            torch.full((d + 8,), -3, dtype=torch.int32, device=dev), torch.zeros(d + 8, dtype=torch.float32, device=dev),
            torch.full((n_segs + 1,), -3, dtype=torch.int32, device=dev))


@pytest.mark.parametrize("sid,max_stages", [(0, 3), (1, -1), (2, -3)])
def test_static_entry_matches_allocating_entry_on_two_calls(sid, max_stages):
    import torch
    from paper_2101_10761_b200 import binding as B
    dev = "cuda:0"
    wl = W.config(2)                       # 269,722 elements in 20 segments, within the static limits
    off, d, S = wl.seg_offsets, wl.d, wl.n_segs
    assert d <= B.STATIC_MAX_ELEMS and S <= B.STATIC_MAX_SEGS
    delta = f32(0.01)
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


def test_static_entry_rekeys_the_shared_array_between_pairs():
    """Two residual buffers and two segment tables take turns on the one array.  Every switch must start
    the incoming pair from a fresh state (M = 1, no counts, no candidate thresholds of the other table),
    which is checked against the oracle restarted at the same moments; within a pair the adaptation runs
    past its first adaptation point (Q = 5).  One table has an empty segment and a one-element segment,
    and one buffer pair is not 32-byte aligned (scalar path)."""
    import torch
    from paper_2101_10761_b200 import binding as B
    dev = "cuda:0"
    tables = [W.offsets_from_sizes([40000, 0, 1, 2500, 70001]), W.offsets_from_sizes([9000, 123457, 31])]
    pairs = [(0, 0, 0), (1, 1, 3), (0, 1, 0)]          # (residual buffer, table, element shift of the pointers)
    delta, sid, ms = f32(0.01), O.SID_EXP, 3
    bufs = {}
    for p, (rb, tb, shift) in enumerate(pairs):
        off = tables[tb]
        bufs[p] = _buffers(int(off[-1]), off.size - 1, dev, shift)
    seed = 500
    for round_ in range(2):
        for p, (rb, tb, shift) in enumerate(pairs):
            off = tables[tb]
            d, S = int(off[-1]), off.size - 1
            sizes = np.diff(off).tolist()
            g_s, r_s, i_s, v_s, k_s = bufs[p]
            # the pair comes back to an array another pair has used since: its state starts over, and so
            # does the residual the test feeds it
            r_s.zero_()
            state, res_o = O.new_state(S), np.zeros(d, np.float32)
            for call in range(7):
                g = W.ragged_case(seed, sizes, 1e-3)
                seed += 1
                g_s.copy_(torch.from_numpy(g))
                B.sidco_compress_static(g_s, r_s, off, delta, sid, ms, i_s, v_s, k_s)
                torch.cuda.synchronize()
                ora = O.sidco_compress(g, res_o, off, delta, sid, ms, state=state)
                out_k = k_s.cpu().numpy()
                k = int(out_k[-1])
                assert np.array_equal(out_k, ora.out_k), (round_, p, call)
                assert np.array_equal(i_s[:k].cpu().numpy(), ora.idx)
                assert np.array_equal(v_s[:k].cpu().numpy().view(np.uint32), ora.val.view(np.uint32))
                assert np.array_equal(r_s.cpu().numpy().view(np.uint32), ora.residual.view(np.uint32))
                res_o = ora.residual
            assert any(st.M > 1 for st in state) or all(st.calls == 7 for st in state)


def test_static_entry_refuses_to_rebuild_under_capture():
    """A (residual, table) pair the array does not hold yet needs uploads and a synchronisation; while the
    stream is capturing the call must return SIDCO_E_CAPTURE and enqueue nothing, and the pair the array
    does hold must keep working afterwards."""
    import torch
    from paper_2101_10761_b200 import binding as B
    dev = "cuda:0"
    off_a, off_b = W.offsets_from_sizes([30000, 500]), W.offsets_from_sizes([12345])
    g_a, r_a, i_a, v_a, k_a = _buffers(int(off_a[-1]), 2, dev)
    g_b, r_b, i_b, v_b, k_b = _buffers(int(off_b[-1]), 1, dev)
    delta = f32(0.01)
    ga = W.ragged_case(900, [30000, 500], 1e-3)
    g_a.copy_(torch.from_numpy(ga))
    B.sidco_compress_static(g_a, r_a, off_a, delta, 0, -1, i_a, v_a, k_a)          # the array now holds pair A
    torch.cuda.synchronize()
    launches = B.sidco_launch_count()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        graph.capture_begin()
        with pytest.raises(B.SidcoError) as err:
            B.sidco_compress_static(g_b, r_b, off_b, delta, 0, -1, i_b, v_b, k_b)
        graph.capture_end()
    assert err.value.code == -11
    assert B.sidco_launch_count() == launches
    torch.cuda.synchronize()
    # pair A carries on from the residual its first call left
    res_o = O.sidco_compress(ga, np.zeros(int(off_a[-1]), np.float32), off_a, delta, 0, -1).residual
    ga2 = W.ragged_case(901, [30000, 500], 1e-3)
    g_a.copy_(torch.from_numpy(ga2))
    B.sidco_compress_static(g_a, r_a, off_a, delta, 0, -1, i_a, v_a, k_a)
    torch.cuda.synchronize()
    ora = O.sidco_compress(ga2, res_o, off_a, delta, 0, -1)
    k = int(k_a[-1])
    assert np.array_equal(k_a.cpu().numpy(), ora.out_k)
    assert np.array_equal(i_a[:k].cpu().numpy(), ora.idx)
    assert np.array_equal(r_a.cpu().numpy().view(np.uint32), ora.residual.view(np.uint32))


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
