"""sidco_compress_bf16: bf16 gradient in, fp32 error-compensation memory.  The oracle gets the same
gradient widened exactly to fp32; everything else is the ordinary parity check."""
import numpy as np
import pytest

from oracle import sidco_oracle as O
from paper_2101_10761_b200 import workloads as W
from parity_util import check_parity, f32

pytestmark = pytest.mark.gpu


def to_bf16_bits(x):
    import torch
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def run_case(sizes, sid, ms, delta, calls, shift=0, scale=1e-3, seed=0):
    import torch
    from paper_2101_10761_b200 import binding as B
    dev = "cuda:0"
    off = W.offsets_from_sizes(sizes)
    d, S = int(off[-1]), len(sizes)
    g_store = torch.zeros(d + 24, dtype=torch.int16, device=dev)
    r_store = torch.zeros(d + 24, dtype=torch.float32, device=dev)
    grad, res = g_store[shift:shift + d], r_store[shift:shift + d]
    out_idx = torch.full((d + 8,), -7, dtype=torch.int32, device=dev)
    out_val = torch.zeros(d + 8, dtype=torch.float32, device=dev)
    out_k = torch.full((S + 1,), -7, dtype=torch.int32, device=dev)
    state = O.new_state(S) if ms > 0 else None
    res_o = np.zeros(d, np.float32)
    key = res.data_ptr() if d else r_store.data_ptr()
    try:
        for call in range(calls):
            bits = to_bf16_bits(W.ragged_case(seed + call, sizes, scale))
            grad.copy_(torch.from_numpy(bits.view(np.int16)))
            B.sidco_compress_bf16(grad.data_ptr() if d else g_store.data_ptr(), key, off, delta, sid, ms,
                                  out_idx, out_val, out_k)
            torch.cuda.synchronize()
            ora = O.sidco_compress(O.bf16_bits_to_f32(bits), res_o, off, delta, sid, ms, state=state)
            ok = out_k.cpu().numpy()
            k = int(ok[-1])
            gpu = dict(idx=out_idx[:k].cpu().numpy(), val=out_val[:k].cpu().numpy(), out_k=ok,
                       residual=res.cpu().numpy(), debug=B.sidco_get_debug(key, S))
            check_parity(gpu, ora, off, state)
            res_o = ora.residual
    finally:
        B.sidco_release(key)


@pytest.mark.parametrize("sid", [0, 1, 2])
@pytest.mark.parametrize("ms", [-1, -3, 4])
def test_resnet20_shaped_bf16(sid, ms):
    run_case(W.config(2).seg_sizes, sid, ms, f32(0.01), 7)


@pytest.mark.parametrize("shift", [0, 1, 4, 8])
def test_ragged_sizes_and_unaligned_pointers(shift):
    run_case([0, 1, 3, 31, 32, 33, 64, 1000, 8191, 8192, 8193, 20000], 2, -2, f32(0.02), 3, shift=shift)


def test_several_million_elements_span_many_runs():
    run_case([3_000_017, 5, 1_500_000], 0, 4, f32(0.001), 6, scale=1e-2)


def test_mixing_fp32_and_bf16_calls_on_one_residual():
    import torch
    from paper_2101_10761_b200 import binding as B
    dev = "cuda:0"
    sizes = [50000, 777]
    off = W.offsets_from_sizes(sizes)
    d, S = int(off[-1]), 2
    res = torch.zeros(d, dtype=torch.float32, device=dev)
    out_idx = torch.empty(d, dtype=torch.int32, device=dev)
    out_val = torch.empty(d, dtype=torch.float32, device=dev)
    out_k = torch.zeros(S + 1, dtype=torch.int32, device=dev)
    res_o, state = np.zeros(d, np.float32), O.new_state(S)
    try:
        for call in range(6):
            g = W.ragged_case(60 + call, sizes, 1e-3)
            if call % 2:
                bits = to_bf16_bits(g)
                g = O.bf16_bits_to_f32(bits)
                B.sidco_compress_bf16(torch.from_numpy(bits.view(np.int16)).to(dev), res, off, f32(0.01), 0, 3,
                                      out_idx, out_val, out_k)
            else:
                B.sidco_compress(torch.from_numpy(g).to(dev), res, off, f32(0.01), 0, 3, out_idx, out_val, out_k)
            torch.cuda.synchronize()
            ora = O.sidco_compress(g, res_o, off, f32(0.01), 0, 3, state=state)
            ok = out_k.cpu().numpy()
            k = int(ok[-1])
            gpu = dict(idx=out_idx[:k].cpu().numpy(), val=out_val[:k].cpu().numpy(), out_k=ok,
                       residual=res.cpu().numpy(), debug=B.sidco_get_debug(res, S))
            check_parity(gpu, ora, off, state)
            res_o = ora.residual
    finally:
        B.sidco_release(res)
