"""Host logic of the sparse exchange (variable-length lists, padding, counts) with two gloo ranks on CPU,
followed by the aggregation oracle on what every rank received."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import os, sys, json
sys.path.insert(0, %r)
import numpy as np, torch, torch.distributed as dist
from paper_2101_10761_b200.exchange import gather_sparse
from oracle import aggregate_oracle as A
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, world = dist.get_rank(), dist.get_world_size()
d = 1000
lists = [(np.array([1, 5, 900], np.int32), np.array([1.0, -2.0, 4.0], np.float32)),
         (np.array([5, 6, 7, 8, 9, 10, 11, 12, 13, 999], np.int32), np.arange(10, dtype=np.float32))]
idx, val = lists[rank]
cap = 64
out_idx = torch.full((cap,), -1, dtype=torch.int32); out_idx[:idx.size] = torch.from_numpy(idx)
out_val = torch.full((cap,), 9.0); out_val[:val.size] = torch.from_numpy(val)
idx_all, val_all, counts, stride = gather_sparse(out_idx, out_val, idx.size)
assert counts.tolist() == [3, 10] and stride == 16 and idx_all.numel() == world * stride
got_lists = [(idx_all[w * stride:w * stride + counts[w]].numpy(), val_all[w * stride:w * stride + counts[w]].numpy())
             for w in range(world)]
for (gi, gv), (wi, wv) in zip(got_lists, lists):
    assert np.array_equal(gi, wi) and np.array_equal(gv, wv)
assert int(idx_all[3]) == 0 and float(val_all[3]) == 0.0            # padding is zeros, not stale buffer contents
dense = A.aggregate([g[0] for g in got_lists], [g[1] for g in got_lists], d)
# fixed-size buffers: a stride the caller chose
_, _, _, s2 = gather_sparse(out_idx, out_val, idx.size, stride=32)
try:
    gather_sparse(out_idx, out_val, idx.size, stride=8)
    small = False
except ValueError:
    small = True
dist.barrier()
print(json.dumps({"rank": rank, "sum": float(dense.sum()), "at5": float(dense[5]), "stride2": s2, "small": small}))
dist.destroy_process_group()
''' % ROOT


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_ranks_exchange_lists_of_different_length():
    port = str(free_port())
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=port)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, cwd=ROOT, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    recs = []
    for p in procs:
        out, err = p.communicate(timeout=600)
        assert p.returncode == 0, err[-3000:]
        recs.append(json.loads(out.strip().splitlines()[-1]))
    for rec in recs:
        assert rec["at5"] == -1.0                   # (-2 + 0) / 2
        assert rec["sum"] == (1.0 - 2.0 + 4.0 + 45.0) / 2
        assert rec["stride2"] == 32 and rec["small"]


def test_single_process_is_a_copy():
    import numpy as np
    import torch
    sys.path.insert(0, ROOT)
    from paper_2101_10761_b200.exchange import gather_sparse
    idx = torch.tensor([2, 4, 6, 0, 0], dtype=torch.int32)
    val = torch.tensor([1.0, 2.0, 3.0, 9.0, 9.0])
    idx_all, val_all, counts, stride = gather_sparse(idx, val, 3)
    assert stride == 8 and counts.tolist() == [3]
    assert idx_all.tolist() == [2, 4, 6, 0, 0, 0, 0, 0] and val_all.tolist()[:4] == [1.0, 2.0, 3.0, 0.0]
