"""Calls recorded by stream capture and replayed as a CUDA graph give the results of the same calls made
directly: the per-call counters live in the workspace, not in the launch arguments."""
import numpy as np
import pytest

from oracle import sidco_oracle as O
from paper_2101_10761_b200 import workloads as W
from parity_util import check_parity, f32

pytestmark = pytest.mark.gpu


def _buffers(torch, d, S):
    dev = "cuda:0"
    return (torch.empty(d + 8, dtype=torch.int32, device=dev), torch.empty(d + 8, dtype=torch.float32, device=dev),
            torch.zeros(S + 1, dtype=torch.int32, device=dev))


def _take(bufs):
    gi, gv, gk = bufs
    out_k = gk.cpu().numpy()
    k = int(out_k[-1])
    return gi[:k].cpu().numpy(), gv[:k].cpu().numpy(), out_k


@pytest.mark.parametrize("sid,ms", [(0, 4), (2, 3)])
def test_graph_replay_matches_direct_calls_and_oracle(sid, ms):
    import torch
    from paper_2101_10761_b200 import binding as B
    wl = W.config(2)
    d, S, off = wl.d, wl.n_segs, wl.seg_offsets
    delta, n_calls = f32(1e-2), 7            # more than Q = 5 calls: the stage adaptation acts inside the run
    grads = [torch.from_numpy(wl.draw(c)).to("cuda:0") for c in range(n_calls)]
    res = torch.zeros(d, dtype=torch.float32, device="cuda:0")
    scratch = _buffers(torch, d, S)
    per_call = [_buffers(torch, d, S) for _ in range(n_calls)]

    # a call under capture before any direct call would have to allocate: refused, nothing enqueued
    side = torch.cuda.Stream()
    g0 = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        g0.capture_begin()
        with pytest.raises(B.SidcoError) as err:
            B.sidco_compress(grads[0], res, off, delta, sid, ms, *scratch)
        g0.capture_end()
    assert err.value.code == -11
    torch.cuda.synchronize()

    # direct run: reset + n_calls calls, checked against the oracle call by call
    B.sidco_compress(grads[0], res, off, delta, sid, ms, *scratch)      # first call: allocates, uploads
    B.sidco_reset_state_async(res)
    state, r_o = O.new_state(S), np.zeros(d, dtype=np.float32)
    direct = []
    for c in range(n_calls):
        B.sidco_compress(grads[c], res, off, delta, sid, ms, *per_call[c])
        torch.cuda.synchronize()
        idx, val, out_k = _take(per_call[c])
        ora = O.sidco_compress(grads[c].cpu().numpy(), r_o, off, delta, sid, ms, state)
        gpu = dict(idx=idx, val=val, out_k=out_k, residual=res.cpu().numpy(), debug=B.sidco_get_debug(res, S))
        check_parity(gpu, ora, off, state)
        r_o = gpu["residual"]
        direct.append((idx, val, out_k))
    final_residual = res.cpu().numpy()

    # the same run recorded once ...
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        graph.capture_begin()
        B.sidco_reset_state_async(res)
        for c in range(n_calls):
            B.sidco_compress(grads[c], res, off, delta, sid, ms, *per_call[c])
        graph.capture_end()
    torch.cuda.synchronize()

    # ... and replayed: every replay starts from the reset and must reproduce the direct run bit for bit
    for replay in range(3):
        res.fill_(float(replay))             # contents must not matter: the reset declares the residual empty
        for bufs in per_call:
            bufs[2].fill_(-1)
        graph.replay()
        torch.cuda.synchronize()
        for c in range(n_calls):
            idx, val, out_k = _take(per_call[c])
            assert np.array_equal(out_k, direct[c][2]), f"replay {replay} call {c}: counts differ"
            assert np.array_equal(idx, direct[c][0])
            assert np.array_equal(val.view(np.uint32), direct[c][1].view(np.uint32))
        assert np.array_equal(res.cpu().numpy().view(np.uint32), final_residual.view(np.uint32))

    # a direct call after the replays carries on from the state the graph left
    B.sidco_compress(grads[0], res, off, delta, sid, ms, *scratch)
    torch.cuda.synchronize()
    idx, val, out_k = _take(scratch)
    ora = O.sidco_compress(grads[0].cpu().numpy(), final_residual, off, delta, sid, ms, state)
    gpu = dict(idx=idx, val=val, out_k=out_k, residual=res.cpu().numpy(), debug=B.sidco_get_debug(res, S))
    check_parity(gpu, ora, off, state)
    B.sidco_release(res)
