"""Exchange of the workers' sparse gradients (plumbing around ``torch.distributed``; no arithmetic).

After ``sidco_compress`` every data-parallel worker holds its own ascending ``(index, value)`` list of
``k_hat`` entries, a different ``k_hat`` on every worker.  ``gather_sparse`` brings all lists to every
worker as three dense buffers that ``sidco_aggregate`` takes: the lists padded to a common stride, and
the counts.  Two collectives: a tiny all-gather of the counts (needed on the host to size the padded
buffers) and one all-gather of the padded lists.  Works with any backend (NCCL on GPUs, gloo in the CPU
tests); with one process it degenerates to a copy.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch


def gather_sparse(out_idx: torch.Tensor, out_val: torch.Tensor, k_hat: int, group=None,
                  stride: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor, int]:
    """All-gather this worker's first ``k_hat`` entries of (out_idx, out_val).

    Returns (idx_all [N * stride] int32, val_all [N * stride] float32, counts [N] int32, stride), worker n's
    list at offset n * stride.  ``stride`` defaults to the largest count rounded up to a multiple of 8
    (at least 8); a caller that wants fixed-size buffers passes its own, which must cover every count."""
    import torch.distributed as dist
    dev = out_idx.device
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    mine = torch.tensor([int(k_hat)], dtype=torch.int32, device=dev)
    if world > 1:
        counts = torch.empty(world, dtype=torch.int32, device=dev)
        dist.all_gather_into_tensor(counts, mine, group=group)
    else:
        counts = mine.clone()
    largest = int(counts.max().item())
    if stride is None:
        stride = max(8, (largest + 7) // 8 * 8)
    elif stride < largest:
        raise ValueError(f"stride {stride} is smaller than the largest list ({largest})")
    pad_idx = torch.zeros(stride, dtype=torch.int32, device=dev)
    pad_val = torch.zeros(stride, dtype=torch.float32, device=dev)
    pad_idx[:k_hat] = out_idx[:k_hat]
    pad_val[:k_hat] = out_val[:k_hat]
    if world > 1:
        idx_all = torch.empty(world * stride, dtype=torch.int32, device=dev)
        val_all = torch.empty(world * stride, dtype=torch.float32, device=dev)
        dist.all_gather_into_tensor(idx_all, pad_idx, group=group)
        dist.all_gather_into_tensor(val_all, pad_val, group=group)
    else:
        idx_all, val_all = pad_idx, pad_val
    return idx_all, val_all, counts, stride
