"""The N > 1 path of the benchmark on CPU: two gloo ranks, independent replicas, MAX of the times
and SUM of the token counts (there is no data-path collective to test)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_23163_b200 import replicas, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = replicas.replica_workload(synth.workload("tiny"), rank)
        pk, _ = synth.make_prefix(w, 0)
        ms = replicas.max_over_ranks(10.0 + 5.0 * rank, dist)            # rank 1 is the slow one
        toks = replicas.sum_over_ranks(12 * (rank + 1), dist)
        out[rank] = (w.seed, int(pk[:4].astype(np.int64).sum()), ms, toks)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_reduce_time_with_max_and_tokens_with_sum():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] != res[1][0]                 # different scenes ...
    assert res[0][1] != res[1][1]                 # ... with different prefix caches
    assert res[0][2] == res[1][2] == 15.0         # every rank sees the slowest rank's time
    assert res[0][3] == res[1][3] == 36.0


def test_without_a_process_group_the_helpers_are_identities():
    w = synth.workload("tiny")
    assert replicas.replica_workload(w, 0) is w
    assert replicas.max_over_ranks(3.5) == 3.5 and replicas.sum_over_ranks(7) == 7.0


def test_bench_gpus_flag_starts_the_ranks_itself():
    # `python bench.py --gpus 2` without a launcher re-executes itself as two ranks; here the ranks only
    # do the bookkeeping (gloo, no GPU): MAX of the times 10 and 11 ms, SUM of 2 x 12 x steps tokens
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--selftest-replicas",
                          "--steps", "5", "--warmup", "3"], capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(x) for x in res.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1                                    # rank 0 alone prints
    line = lines[0]
    assert line["n_gpus"] == 2 and line["steps"] == 5 and line["warmup"] == 3
    assert abs(line["ms_per_step"] - 11.0 / 5) < 1e-12
    assert abs(line["value"] - 120.0 / 11e-3) < 1e-6
