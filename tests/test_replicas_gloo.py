"""The N > 1 path of bench.py on CPU: two gloo ranks draw distinct batches, agree on the slowest
rank's time and report the whole-job rate (replicas only: no data-path collective)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from synth_inputs import WORKLOADS, make_hidden


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = bench.rank_workload(WORKLOADS["tiny"], rank)
        h = make_hidden(w, 0)
        ms_local = 10.0 * (rank + 1)                      # rank 1 is the slow one
        ms_max = bench.max_over_ranks(ms_local)
        val = bench.whole_job_tokens_per_s(world, w.T, ms_max)
        sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sums, torch.tensor([float(h.astype(np.float64).sum())], dtype=torch.float64))
        out[rank] = (ms_max, val, [float(x) for x in sums])
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_max_time_and_distinct_batches():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for r in (0, 1):
        ms_max, val, sums = res[r]
        assert ms_max == 20.0                             # the max over ranks, on every rank
        assert abs(val - 2 * WORKLOADS["tiny"].T / 0.020) < 1e-6
        assert sums[0] != sums[1]                         # distinct data per replica
    assert res[0][2] == res[1][2]


def test_single_rank_helpers_are_identity():
    assert bench.max_over_ranks(12.5) == 12.5
    assert bench.rank_workload(WORKLOADS["mid"], 0) is WORKLOADS["mid"]
    assert bench.rank_workload(WORKLOADS["mid"], 3).seed != WORKLOADS["mid"].seed
