"""The path does not shard: N GPUs run N independent replicas.  These CPU tests cover the host logic
of that mode with two gloo ranks: the cross-rank reduction bench.py uses (max of times, sum of work)
and the rule that only rank 0 runs the reference arm."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import os, sys, json
sys.path.insert(0, %r)
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank = dist.get_rank()
times, totals = bench.reduce_over_ranks(dist, torch.device("cpu"), [10.0 + rank, 3.0 - rank], [100.0, 7.0 * (rank + 1)])
dist.barrier()
print(json.dumps({"rank": rank, "times": times, "totals": totals}))
dist.destroy_process_group()
'''


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch(code_or_args, world=2, as_code=True):
    port = str(free_port())
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=port)
        cmd = [sys.executable, "-c", code_or_args] if as_code else [sys.executable] + code_or_args
        procs.append(subprocess.Popen(cmd, env=env, cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=600)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_reduction_is_max_of_times_and_sum_of_work():
    outs = launch(WORKER % ROOT)
    for out in outs:
        rec = json.loads(out.strip().splitlines()[-1])
        assert rec["times"] == [11.0, 3.0]          # max over ranks, entry by entry
        assert rec["totals"] == [200.0, 21.0]       # sum over ranks


def test_single_process_reduction_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(None, None, [1.5, 2.5], [3, 4]) == ([1.5, 2.5], [3, 4])


def test_reference_arm_runs_on_rank_zero_only():
    outs = launch([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "2", "--warmup", "3"],
                  as_code=False)
    assert outs[1].strip() == ""
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0
