"""The Ring-DTP schedule across ranks (Algorithm 3, both branches), run as gloo ranks on the CPU with a float64
stand-in for the CUDA meetings.  Checked against the oracle's dense definition on the group's global problem:
every (batch, shard) pair is met exactly once in the order q = (r - i) mod P, the travelling state / gradient
arrives where it belongs (dW_q back at its owner, per-token results and dX back at the batch's rank), and the
auto rule picks move-weights exactly when N > V / P."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import vpce_oracle as orc
from paper_2609_14306_b200 import ring
from ring_testlib import OracleMeetings, global_problem

IGNORE = -100


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, cfg, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        N, d, V, mode, seed = cfg
        X, W, t = global_problem(world, N, d, V, seed)
        lo, hi = ring.shard_interval(rank, V, world)
        Xr = torch.from_numpy(X[rank * N:(rank + 1) * N]).float()
        tr = torch.from_numpy(t[rank * N:(rank + 1) * N])
        Wr = torch.from_numpy(W[lo:hi]).float()
        log = []
        drv = ring.RingDTP(ring.DistTransport(), V, d, IGNORE, mode=mode, meetings=OracleMeetings(), log=log)
        loss, lse = drv.forward(Xr, tr, Wr)
        dloss = drv.masked_mean_dloss(tr)
        dX, dW = drv.backward(Xr, tr, Wr, lse, dloss)
        # a second backward accumulates into the same buffer
        dX2, dW2 = drv.backward(Xr, tr, Wr, lse, dloss, dW_own=dW.clone(), accumulate_dW=True)
        out[rank] = dict(loss=loss.numpy(), lse=lse.numpy(), dloss=dloss.numpy(), dX=dX.numpy(), dW=dW.numpy(),
                         dW2=dW2.numpy(), dX2=dX2.numpy(), log=log, schedule=drv.schedule(N))
    finally:
        dist.destroy_process_group()


def _run(world, cfg):
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, cfg, out), nprocs=world, join=True)
        return dict(out)


@pytest.mark.parametrize("world,N,d,V,mode,expect", [
    (2, 64, 16, 96, "auto", "weights"),          # N = 64 > V/P = 48
    (2, 40, 16, 96, "auto", "activations"),      # N = 40 <= 48
    (3, 24, 8, 100, "weights", "weights"),       # V not divisible by P: shards of 34, 34, 32 rows
    (3, 24, 8, 100, "activations", "activations"),
    (4, 16, 8, 64, "auto", "activations"),       # N = V/P exactly: the rule is a strict inequality
    (4, 20, 8, 64, "auto", "weights"),
])
def test_ring_schedule_matches_the_dense_definition(world, N, d, V, mode, expect):
    res = _run(world, (N, d, V, mode, 1000 + world * 7 + N))
    assert set(res) == set(range(world))
    X, W, t = global_problem(world, N, d, V, 1000 + world * 7 + N)
    dl = orc.default_dloss(t, IGNORE)
    ref = orc.forward_backward(X.astype(np.float32).astype(np.float64), W.astype(np.float32).astype(np.float64), t, dl, IGNORE)
    pairs = {"fwd": [], "bwd": []}
    for r in range(world):
        o = res[r]
        sl = slice(r * N, (r + 1) * N)
        lo, hi = ring.shard_interval(r, V, world)
        assert o["schedule"] == expect
        np.testing.assert_allclose(o["lse"], ref["lse"][sl], rtol=0, atol=2e-5)
        np.testing.assert_allclose(o["loss"], ref["loss"][sl], rtol=0, atol=2e-5)
        np.testing.assert_allclose(o["dloss"], dl[sl], rtol=1e-6, atol=0)          # 1 / n_valid of the WHOLE group
        assert np.linalg.norm(o["dX"] - ref["dH"][sl]) <= 1e-5 * np.linalg.norm(ref["dH"][sl])
        assert np.linalg.norm(o["dW"] - ref["dW"][lo:hi]) <= 1e-5 * np.linalg.norm(ref["dW"][lo:hi])
        assert np.linalg.norm(o["dW2"] - 2 * ref["dW"][lo:hi]) <= 1e-5 * np.linalg.norm(2 * ref["dW"][lo:hi])
        np.testing.assert_array_equal(o["dX2"], o["dX"])
        # the order of the meetings on this rank
        for what in ("fwd", "bwd"):
            seq = [(i, owner, q) for (w_, i, owner, q) in o["log"] if w_ == what][:world]
            assert [i for i, _, _ in seq] == list(range(world))
            if expect == "weights":
                assert [q for _, _, q in seq] == orc.shard_order(r, world)           # q = (r - i) mod P
                assert all(owner == r for _, owner, _ in seq)
            else:
                assert [owner for _, owner, _ in seq] == orc.shard_order(r, world)   # batch of rank (r - i) mod P
                assert all(q == r for _, _, q in seq)
            pairs[what] += [(owner, q) for _, owner, q in seq]
    for what in ("fwd", "bwd"):
        assert sorted(pairs[what]) == [(j, q) for j in range(world) for q in range(world)]   # each pair exactly once


def test_rule_and_intervals():
    assert ring.choose_schedule(32768, 200000, 8) == "weights"        # the paper's Table 2 rows
    assert ring.choose_schedule(16384, 200000, 8) == "activations"
    assert ring.choose_schedule(25000, 200000, 8) == "activations"    # N == V / P: weights move only if N > V / P
    assert [ring.shard_interval(q, 100, 3) for q in range(3)] == [(0, 34), (34, 68), (68, 100)]
    assert ring.shard_interval(7, 200000, 8) == (175000, 200000)


def test_single_rank_group_needs_no_process_group():
    class Solo:
        rank, size = 0, 1

        def exchange(self, send, recv):
            for s, r in zip(send, recv):
                r.copy_(s)
            return type("H", (), {"wait": lambda self: None})()

        def all_sum(self, v):
            return v

    N, d, V = 12, 8, 40
    X, W, t = global_problem(1, N, d, V, 5)
    ref = orc.forward_backward(X.astype(np.float32).astype(np.float64), W.astype(np.float32).astype(np.float64), t, None, IGNORE)
    for mode in ("weights", "activations"):
        drv = ring.RingDTP(Solo(), V, d, IGNORE, mode=mode, meetings=OracleMeetings())
        Xr, tr, Wr = torch.from_numpy(X).float(), torch.from_numpy(t), torch.from_numpy(W).float()
        loss, lse = drv.forward(Xr, tr, Wr)
        dX, dW = drv.backward(Xr, tr, Wr, lse, drv.masked_mean_dloss(tr))
        np.testing.assert_allclose(lse.numpy(), ref["lse"], atol=2e-5)
        assert np.linalg.norm(dX.numpy() - ref["dH"]) <= 1e-5 * np.linalg.norm(ref["dH"])
        assert np.linalg.norm(dW.numpy() - ref["dW"]) <= 1e-5 * np.linalg.norm(ref["dW"])
