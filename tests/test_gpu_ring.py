"""The ring driver with the real CUDA meetings, on ONE GPU: the P ranks of a projection group run as P host
threads of this process, each with its own driver, batch and shard, and hand tensors to one another through
host-side queues (a copy that is finished before it is handed over), so no kernel ever waits for another one.
Results are compared with the float64 oracle on the group's global problem.  What this cannot cover is the NCCL
transport itself; the same schedule runs over gloo ranks in test_ring_gloo.py."""
import queue
import threading

import numpy as np
import pytest
import torch

from oracle import vpce_oracle as orc
from paper_2609_14306_b200 import ring
from synth_inputs import IGNORE_INDEX, bf16_bits_to_f64, f32_to_bf16_bits
from vpce_testlib import TOL_GRAD, TOL_TOKEN, relF, to_dev_bf16

pytestmark = pytest.mark.gpu


class ThreadTransport:
    """Ring of host threads: `exchange` hands finished copies to the next rank's queue; `wait` takes what the
    previous rank handed over and copies it into the receive buffers."""

    def __init__(self, rank, size, queues, shared=None):
        self.rank, self.size, self.queues, self.shared = rank, size, queues, shared

    def exchange(self, send, recv):
        copies = [s.clone() for s in send]
        torch.cuda.current_stream().synchronize()            # the copies are complete before anyone sees them
        self.queues[(self.rank + 1) % self.size].put(copies)
        tp = self

        class Handle:
            def wait(self_inner):
                got = tp.queues[tp.rank].get(timeout=120)
                assert len(got) == len(recv)
                for g, r in zip(got, recv):
                    r.copy_(g)
        return Handle()

    def all_sum(self, value):
        slots, barrier = self.shared
        slots[self.rank] = int(value)
        barrier.wait(timeout=120)
        total = sum(slots)
        barrier.wait(timeout=120)                             # nobody overwrites a slot before all have read
        return total


def _problem(P, N, d, V, seed):
    rng = np.random.default_rng(seed)
    Xb = f32_to_bf16_bits(rng.standard_normal((P * N, d)).astype(np.float32))
    Wb = f32_to_bf16_bits((rng.standard_normal((V, d)) / np.sqrt(d)).astype(np.float32))
    t = rng.integers(0, V, size=P * N).astype(np.int32)
    t[rng.random(P * N) < 0.08] = IGNORE_INDEX
    t[0], t[-1] = 0, V - 1
    return Xb, Wb, t


@pytest.mark.parametrize("P,N,d,V,mode", [
    (2, 256, 256, 1500, "weights"),          # shards of 750 rows: not a multiple of the vocabulary tile
    (2, 256, 256, 1500, "activations"),
    (3, 384, 128, 2000, "weights"),          # shards of 667, 667, 666 rows
    (3, 130, 128, 2000, "activations"),      # a batch that ends inside a token tile (one-CTA kernels + ragged rows)
    (1, 256, 64, 700, "weights"),
])
def test_ring_threads_on_one_gpu_match_the_oracle(P, N, d, V, mode):
    Xb, Wb, t = _problem(P, N, d, V, seed=P * 100 + N)
    X64, W64 = bf16_bits_to_f64(Xb), bf16_bits_to_f64(Wb)
    dl = orc.default_dloss(t, IGNORE_INDEX)
    ref = orc.forward_backward(X64, W64, t, dl, IGNORE_INDEX)
    queues = [queue.Queue() for _ in range(P)]
    out, errors = {}, []

    def rank_main(r):
        try:
            lo, hi = ring.shard_interval(r, V, P)
            Xr = to_dev_bf16(Xb[r * N:(r + 1) * N])
            Wr = to_dev_bf16(Wb[lo:hi])
            tr = torch.from_numpy(t[r * N:(r + 1) * N]).cuda()
            dlr = torch.from_numpy(dl[r * N:(r + 1) * N].astype(np.float32)).cuda()
            log = []
            drv = ring.RingDTP(ThreadTransport(r, P, queues), V, d, IGNORE_INDEX, mode=mode, log=log)
            loss, lse = drv.forward(Xr, tr, Wr)
            dX, dW = drv.backward(Xr, tr, Wr, lse, dlr)
            torch.cuda.synchronize()
            out[r] = (loss.cpu().numpy(), lse.cpu().numpy(), dX.float().cpu().numpy(), dW.cpu().numpy(), log)
        except Exception as exc:                              # surfaced by the main thread
            errors.append((r, repr(exc)))

    threads = [threading.Thread(target=rank_main, args=(r,)) for r in range(P)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=300)
    assert not errors, errors
    assert set(out) == set(range(P))
    dW_all = np.zeros((V, d))
    for r in range(P):
        loss, lse, dX, dW, log = out[r]
        sl = slice(r * N, (r + 1) * N)
        lo, hi = ring.shard_interval(r, V, P)
        assert np.abs(lse - ref["lse"][sl]).max() <= TOL_TOKEN
        assert np.abs(loss - ref["loss"][sl]).max() <= TOL_TOKEN
        assert relF(dX, ref["dH"][sl]) <= TOL_GRAD
        assert relF(dW, ref["dW"][lo:hi]) <= TOL_GRAD
        dW_all[lo:hi] = dW
        assert len([1 for w_, *_ in log if w_ == "fwd"]) == P and len([1 for w_, *_ in log if w_ == "bwd"]) == P
    assert relF(dW_all, ref["dW"]) <= TOL_GRAD


@pytest.mark.parametrize("mode", ["weights", "activations"])
def test_ring_mean_loss_gradient_and_accumulation_into_an_existing_dW(mode):
    # the upstream gradient of the group-wide masked mean comes from the library (count + 1/n on valid tokens),
    # and a second backward with accumulate_dW adds to what dW_own already holds
    P, N, d, V = 2, 256, 128, 1100
    Xb, Wb, t = _problem(P, N, d, V, seed=77)
    t[5] = V + 3                                              # an out-of-range target counts as ignored
    X64, W64 = bf16_bits_to_f64(Xb), bf16_bits_to_f64(Wb)
    valid = (t != IGNORE_INDEX) & (t >= 0) & (t < V)
    dl = np.where(valid, 1.0 / valid.sum(), 0.0)
    t_ref = np.where(valid, t, IGNORE_INDEX).astype(np.int32)
    ref = orc.forward_backward(X64, W64, t_ref, dl, IGNORE_INDEX)
    queues = [queue.Queue() for _ in range(P)]
    shared = ([0] * P, threading.Barrier(P))
    out, errors = {}, []

    def rank_main(r):
        try:
            lo, hi = ring.shard_interval(r, V, P)
            Xr = to_dev_bf16(Xb[r * N:(r + 1) * N])
            Wr = to_dev_bf16(Wb[lo:hi])
            tr = torch.from_numpy(t[r * N:(r + 1) * N]).cuda()
            drv = ring.RingDTP(ThreadTransport(r, P, queues, shared), V, d, IGNORE_INDEX, mode=mode)
            loss, lse = drv.forward(Xr, tr, Wr)
            dlr = drv.masked_mean_dloss(tr)
            dX, dW = drv.backward(Xr, tr, Wr, lse, dlr)
            once = dW.clone()
            dX2, dW2 = drv.backward(Xr, tr, Wr, lse, dlr, dW_own=dW, accumulate_dW=True)
            torch.cuda.synchronize()
            out[r] = (dlr.cpu().numpy(), dX.float().cpu().numpy(), once.cpu().numpy(), dW2.cpu().numpy(),
                      dX2.float().cpu().numpy())
        except Exception as exc:
            errors.append((r, repr(exc)))

    threads = [threading.Thread(target=rank_main, args=(r,)) for r in range(P)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=300)
    assert not errors, errors
    for r in range(P):
        dlr, dX, once, twice, dX2 = out[r]
        sl = slice(r * N, (r + 1) * N)
        lo, hi = ring.shard_interval(r, V, P)
        assert np.array_equal(dlr, dl[sl].astype(np.float32))
        assert relF(dX, ref["dH"][sl]) <= TOL_GRAD and np.array_equal(dX, dX2)
        assert relF(once, ref["dW"][lo:hi]) <= TOL_GRAD
        assert relF(twice, 2.0 * ref["dW"][lo:hi]) <= TOL_GRAD


def test_meeting_entry_points_reject_bad_arguments():
    import paper_2609_14306_b200 as vp
    X = torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(256, 64, dtype=torch.bfloat16, device="cuda")
    t = torch.zeros(128, dtype=torch.int32, device="cuda")
    state = torch.zeros(3, 128, device="cuda")
    out = torch.zeros(128, device="cuda")
    ws = torch.empty(vp.vp_ce_meeting_workspace_bytes(128, 64, 256), dtype=torch.uint8, device="cuda")
    with pytest.raises(vp.VpceError) as ei:          # the shard would reach past the vocabulary
        vp.vp_ce_meeting_forward(X, W, t, 900, 1000, IGNORE_INDEX, state, True, True, out, out, ws)
    assert ei.value.code == 1
    with pytest.raises(vp.VpceError) as ei:          # workspace of a smaller meeting
        vp.vp_ce_meeting_forward(X, W, t, 0, 1000, IGNORE_INDEX, state, True, True, out, out, ws[:4096])
    assert ei.value.code == 3
    with pytest.raises(vp.VpceError) as ei:          # an input-gradient phase that is not the first needs its accumulator
        vp.vp_ce_meeting_backward(X, W, t, out, out, 0, 1000, IGNORE_INDEX, vp.PHASE_INPUT_GRAD, None, False, True,
                                  X.clone(), None, False, ws)
    assert ei.value.code == 1
    assert vp.vp_ce_meeting_workspace_bytes(0, 64, 256) == 0
