"""Ring-DTP across devices: the schedule of Algorithm 3 (paper section 3.2, Appendix C) around the per-meeting
CUDA entry points ``vp_ce_meeting_forward`` / ``vp_ce_meeting_backward``.

Rank r of a projection group of size P holds its own batch ``X_r [N, d]`` with targets ``t_r`` and owns the
vocabulary interval ``V_r = [r*S, min(V, (r+1)*S))`` with ``S = ceil(V / P)``, i.e. the rows ``W_r`` of the
projection weight.  Over P rounds every batch meets every shard exactly once; a meeting forms one logit strip,
folds it into the batch's per-token state ``(m, z, y_t)`` and drops it.  Either operand can travel:

* move-weights (chosen when ``N > V / P``): ``(X_r, t_r, S_r)`` stay, the shard held in round i is
  ``q = (r - i) mod P``; it is sent to rank r+1 while the rank computes with it, and the next one is received from
  rank r-1 into a second buffer.  Forward needs no return hop.  In backward the fp32 gradient ``dW_q`` travels
  with its shard and takes one last hop home.
* move-activations (otherwise): the shard stays, ``(X, t, state)`` travel; after the last round the finished
  per-token results take one hop home.  In backward ``(X, t, lse, dloss)`` travel with the fp32 accumulator of
  ``dX``; ``dW_r`` accumulates at home.

This module holds NO arithmetic of the method: every meeting runs in the CUDA library (``CudaMeetings``) or in
whatever object with the same three methods the caller supplies.  Transfers go through a transport object:
``DistTransport`` uses ``torch.distributed`` point-to-point operations (NCCL between GPUs: the received tensor
lands in this rank's own memory and kernels read local memory only).  Read-only operands of round i+1 move while
round i computes; a travelling accumulator is sent as soon as the phase that produced it is enqueued and is waited
for just before the phase that consumes it.

All ranks must call ``forward`` / ``backward`` collectively with the same N.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch

from . import binding as _b

MOVE_WEIGHTS = "weights"
MOVE_ACTIVATIONS = "activations"


def choose_schedule(N: int, V: int, P: int) -> str:
    """The paper's rule: bytes per hop are O(N d) if activations move and O(d V / P) if weights move, so the
    weights move exactly when N > V / P."""
    return MOVE_WEIGHTS if N * P > V else MOVE_ACTIVATIONS


def shard_interval(q: int, V: int, P: int) -> Tuple[int, int]:
    """Vocabulary ids [lo, hi) owned by rank q: contiguous blocks of S = ceil(V / P) rows (the last may be shorter)."""
    S = -(-V // P)
    lo = min(V, q * S)
    return lo, min(V, lo + S)


# ----------------------------------------------------------------------------------------------- transports
class _Handle:
    def __init__(self, works):
        self._works = works

    def wait(self) -> None:
        for w in self._works:
            w.wait()
        self._works = []


class DistTransport:
    """Point-to-point ring over a ``torch.distributed`` process group (NCCL on GPUs, gloo on CPU)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self._dist = dist
        self.group = group
        self.rank = dist.get_rank(group)
        self.size = dist.get_world_size(group)
        to_global = (lambda r: dist.get_global_rank(group, r)) if group is not None else (lambda r: r)
        self._next = to_global((self.rank + 1) % self.size)
        self._prev = to_global((self.rank - 1) % self.size)

    def exchange(self, send: Sequence[torch.Tensor], recv: Sequence[torch.Tensor]) -> _Handle:
        """Starts sending every tensor of `send` to rank r+1 and receiving into every tensor of `recv` from rank
        r-1 (same count, shapes and dtypes on all ranks).  Returns at once; ``wait()`` orders the caller's stream
        (CUDA) or the caller (CPU) after the transfers."""
        if self.size == 1:
            for s, r in zip(send, recv):
                r.copy_(s)
            return _Handle([])
        dist = self._dist
        ops = [dist.P2POp(dist.isend, t, self._next, self.group) for t in send]
        ops += [dist.P2POp(dist.irecv, t, self._prev, self.group) for t in recv]
        return _Handle(dist.batch_isend_irecv(ops))

    def all_sum(self, value: int) -> int:
        t = torch.tensor([int(value)], dtype=torch.int64)
        if self.size > 1:
            backend = self._dist.get_backend(self.group)
            if backend == "nccl":
                t = t.cuda()
            self._dist.all_reduce(t, group=self.group)
        return int(t.item())


# ----------------------------------------------------------------------------------------------- meetings
class CudaMeetings:
    """The meetings as the CUDA library computes them (bf16 operands, fp32 state and accumulators)."""

    operand_dtype = torch.bfloat16

    def workspace(self, N: int, d: int, S: int, device) -> torch.Tensor:
        n = _b.vp_ce_meeting_workspace_bytes(N, d, S)
        if n == 0:
            raise ValueError("shape rejected by vp_ce_meeting_workspace_bytes (d must be a multiple of 8)")
        return torch.empty(n, dtype=torch.uint8, device=device)

    def forward_meeting(self, X, W, t, v_lo, V, ignore_index, state, first, last, loss, lse, ws) -> None:
        _b.vp_ce_meeting_forward(X, W, t, v_lo, V, ignore_index, state, first, last, loss, lse, ws)

    def count_valid(self, t, V, ignore_index) -> int:
        """Number of tokens whose target is neither ignore_index nor outside [0, V) (vp_ce_mean_loss's count)."""
        zeros = torch.zeros(t.numel(), dtype=torch.float32, device=t.device)
        mean = torch.empty(1, dtype=torch.float32, device=t.device)
        n = torch.empty(1, dtype=torch.int32, device=t.device)
        _b.vp_ce_mean_loss(zeros, t, V, ignore_index, mean, n)
        return int(n.item())

    def mean_dloss(self, t, V, ignore_index, n_valid_total: int) -> torch.Tensor:
        """1 / n_valid_total on valid tokens, 0 elsewhere (vp_ce_mean_loss_grad)."""
        n = torch.tensor([int(n_valid_total)], dtype=torch.int32, device=t.device)
        out = torch.empty(t.numel(), dtype=torch.float32, device=t.device)
        _b.vp_ce_mean_loss_grad(t, V, ignore_index, n, None, out)
        return out

    def backward_meeting(self, X, W, t, lse, dloss, v_lo, V, ignore_index, phases, dX_acc, first, last, dX, dW,
                         accumulate_dW, ws) -> None:
        _b.vp_ce_meeting_backward(X, W, t, lse, dloss, v_lo, V, ignore_index, phases, dX_acc, first, last, dX, dW,
                                  accumulate_dW, ws)


# ----------------------------------------------------------------------------------------------- the driver
class RingDTP:
    """Algorithm 3 on rank ``transport.rank`` of a projection group of ``transport.size`` ranks."""

    def __init__(self, transport, V: int, d: int, ignore_index: int = -100, mode: str = "auto", meetings=None,
                 log: Optional[List[tuple]] = None):
        if mode not in ("auto", MOVE_WEIGHTS, MOVE_ACTIVATIONS):
            raise ValueError("mode must be 'auto', 'weights' or 'activations'")
        self.tp = transport
        self.P, self.r = transport.size, transport.rank
        self.V, self.d, self.ignore_index, self.mode = int(V), int(d), int(ignore_index), mode
        self.S = -(-self.V // self.P)
        if shard_interval(self.P - 1, self.V, self.P)[1] - shard_interval(self.P - 1, self.V, self.P)[0] <= 0:
            raise ValueError("V is too small for this group: the last rank would own no vocabulary row")
        self.meetings = meetings if meetings is not None else CudaMeetings()
        self.log = log                     # optional: (pass, round, batch owner, shard) of every meeting, for tests
        self._ws = None

    # ---- helpers
    def schedule(self, N: int) -> str:
        return choose_schedule(N, self.V, self.P) if self.mode == "auto" else self.mode

    def _interval(self, q: int) -> Tuple[int, int]:
        return shard_interval(q, self.V, self.P)

    def _workspace(self, N: int, device) -> torch.Tensor:
        if self._ws is None or self._ws[0] != (N, str(device)):
            self._ws = ((N, str(device)), self.meetings.workspace(N, self.d, self.S, device))
        return self._ws[1]

    def _check(self, X, t, W_own) -> int:
        lo, hi = self._interval(self.r)
        if X.dim() != 2 or X.shape[1] != self.d or t.shape != (X.shape[0],):
            raise ValueError("X must be [N, d] and t [N]")
        if tuple(W_own.shape) != (hi - lo, self.d):
            raise ValueError(f"rank {self.r} owns vocabulary rows [{lo}, {hi}): W_own must be [{hi - lo}, {self.d}]")
        return int(X.shape[0])

    def _note(self, what: str, i: int, owner: int, q: int) -> None:
        if self.log is not None:
            self.log.append((what, i, owner, q))

    def masked_mean_dloss(self, t: torch.Tensor) -> torch.Tensor:
        """Upstream gradient of the mean loss over the valid tokens of ALL ranks' batches: 1 / n_valid_total on
        valid tokens (one integer all-reduce of the local counts; the paper's operator itself outputs per-token
        values).  The counting and the per-token values come from the meetings object (the CUDA library)."""
        total = self.tp.all_sum(self.meetings.count_valid(t, self.V, self.ignore_index))
        return self.meetings.mean_dloss(t, self.V, self.ignore_index, total)

    # ---- forward
    def forward(self, X: torch.Tensor, t: torch.Tensor, W_own: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
        """Per-token (loss, lse) of this rank's batch against the WHOLE vocabulary (Algorithm 3)."""
        N = self._check(X, t, W_own)
        if self.schedule(N) == MOVE_WEIGHTS:
            return self._forward_move_weights(X, t, W_own, N)
        return self._forward_move_activations(X, t, W_own, N)

    def _forward_move_weights(self, X, t, W_own, N):
        P, r, S, dev = self.P, self.r, self.S, X.device
        ws = self._workspace(N, dev)
        state = torch.empty(3, N, dtype=torch.float32, device=dev)
        loss = torch.empty(N, dtype=torch.float32, device=dev)
        lse = torch.empty(N, dtype=torch.float32, device=dev)
        bufs = [torch.empty(S, self.d, dtype=W_own.dtype, device=dev) for _ in range(2 if P > 1 else 1)]
        bufs[0][: W_own.shape[0]].copy_(W_own)
        if W_own.shape[0] < S:
            bufs[0][W_own.shape[0]:].zero_()              # padding rows of the last shard: defined bytes on the wire
        for i in range(P):
            q = (r - i) % P                               # Algorithm 3: q = (r - i) mod P
            cur = bufs[i % 2]
            # the shard travels on while this round computes with it; the next one lands in the other buffer
            moving = self.tp.exchange([cur], [bufs[(i + 1) % 2]]) if i < P - 1 else None
            lo, hi = self._interval(q)
            self.meetings.forward_meeting(X, cur[: hi - lo], t, lo, self.V, self.ignore_index, state, i == 0,
                                          i == P - 1, loss, lse, ws)
            self._note("fwd", i, r, q)
            if moving is not None:
                moving.wait()
        return loss, lse

    def _forward_move_activations(self, X, t, W_own, N):
        P, r, dev = self.P, self.r, X.device
        ws = self._workspace(N, dev)
        lo, _ = self._interval(r)
        nb = 2 if P > 1 else 1
        Xb = [torch.empty_like(X) for _ in range(nb)]
        tb = [torch.empty_like(t) for _ in range(nb)]
        Sb = [torch.empty(3, N, dtype=torch.float32, device=dev) for _ in range(nb)]
        out = [torch.empty(2, N, dtype=torch.float32, device=dev) for _ in range(2)]     # (loss, lse): remote, home
        Xb[0].copy_(X)
        tb[0].copy_(t)
        state_moving = None
        for i in range(P):
            owner = (r - i) % P                           # whose batch is here in round i
            c, n = i % 2, (i + 1) % 2
            ops_moving = self.tp.exchange([Xb[c], tb[c]], [Xb[n], tb[n]]) if i < P - 1 else None
            if state_moving is not None:
                state_moving.wait()                       # this batch's running state, from rank r-1
            self.meetings.forward_meeting(Xb[c], W_own, tb[c], lo, self.V, self.ignore_index, Sb[c], i == 0, i == P - 1,
                                          out[0][0], out[0][1], ws)
            self._note("fwd", i, owner, r)
            state_moving = self.tp.exchange([Sb[c]], [Sb[n]]) if i < P - 1 else None
            if ops_moving is not None:
                ops_moving.wait()
        # the finished results of the batch that ended here go one hop on, those of this rank's batch arrive
        # (Algorithm 3 returns the state and finalises at home; the last meeting finalises here, so two floats per
        # token travel instead of three)
        self.tp.exchange([out[0]], [out[1]]).wait()
        return out[1][0], out[1][1]

    # ---- backward
    def backward(self, X: torch.Tensor, t: torch.Tensor, W_own: torch.Tensor, lse: torch.Tensor, dloss: torch.Tensor,
                 dW_own: Optional[torch.Tensor] = None, accumulate_dW: bool = False):
        """(dX [N, d] in X's dtype, dW_own fp32 [rows of V_r, d]) from the saved normaliser ``lse`` and the
        per-token upstream gradient ``dloss``.  With ``accumulate_dW`` the result is added into ``dW_own``."""
        N = self._check(X, t, W_own)
        if dW_own is None:
            if accumulate_dW:
                raise ValueError("accumulate_dW needs dW_own")
            dW_own = torch.empty(W_own.shape, dtype=torch.float32, device=X.device)
        if self.schedule(N) == MOVE_WEIGHTS:
            return self._backward_move_weights(X, t, W_own, lse, dloss, dW_own, accumulate_dW, N)
        return self._backward_move_activations(X, t, W_own, lse, dloss, dW_own, accumulate_dW, N)

    def _backward_move_weights(self, X, t, W_own, lse, dloss, dW_own, accumulate_dW, N):
        P, r, S, dev = self.P, self.r, self.S, X.device
        ws = self._workspace(N, dev)
        M = self.meetings
        RES_IN, WG = _b.PHASE_RESIDUAL | _b.PHASE_INPUT_GRAD, _b.PHASE_WEIGHT_GRAD
        dX = torch.empty_like(X)
        dX_acc = torch.empty(N, self.d, dtype=torch.float32, device=dev) if P > 1 else None
        Wb = [torch.empty(S, self.d, dtype=W_own.dtype, device=dev) for _ in range(2 if P > 1 else 1)]
        Db = [torch.empty(S, self.d, dtype=torch.float32, device=dev) for _ in range(2)]
        Wb[0][: W_own.shape[0]].copy_(W_own)
        if W_own.shape[0] < S:
            Wb[0][W_own.shape[0]:].zero_()
        for b in Db:
            b.zero_()                                     # padding rows stay zero on the wire
        if accumulate_dW:
            Db[0][: W_own.shape[0]].copy_(dW_own)         # the travelling gradient starts from what the owner holds
        grad_moving = None
        for i in range(P):
            q = (r - i) % P
            c, n = i % 2, (i + 1) % 2
            w_moving = self.tp.exchange([Wb[c]], [Wb[n]]) if i < P - 1 else None
            lo, hi = self._interval(q)
            M.backward_meeting(X, Wb[c][: hi - lo], t, lse, dloss, lo, self.V, self.ignore_index, RES_IN, dX_acc, i == 0,
                               i == P - 1, dX, None, False, ws)
            if grad_moving is not None:
                grad_moving.wait()                        # the partial dW_q of the ranks that met q before this one
            M.backward_meeting(X, Wb[c][: hi - lo], t, lse, dloss, lo, self.V, self.ignore_index, WG, None, i == 0,
                               i == P - 1, None, Db[c][: hi - lo], i > 0 or accumulate_dW, ws)
            self._note("bwd", i, r, q)
            # the gradient travels with its shard; after the last round this hop brings every dW_q home
            grad_moving = self.tp.exchange([Db[c]], [Db[n]])
            if w_moving is not None:
                w_moving.wait()
        grad_moving.wait()
        dW_own.copy_(Db[P % 2][: W_own.shape[0]])           # this rank's own shard is home again, complete
        return dX, dW_own

    def _backward_move_activations(self, X, t, W_own, lse, dloss, dW_own, accumulate_dW, N):
        P, r, dev = self.P, self.r, X.device
        ws = self._workspace(N, dev)
        M = self.meetings
        lo, _ = self._interval(r)
        nb = 2 if P > 1 else 1
        Xb = [torch.empty_like(X) for _ in range(nb)]
        tb = [torch.empty_like(t) for _ in range(nb)]
        Lb = [torch.empty(2, N, dtype=torch.float32, device=dev) for _ in range(nb)]      # (lse, dloss) of the batch
        Ab = [torch.empty(N, self.d, dtype=torch.float32, device=dev) for _ in range(nb)] if P > 1 else [None]
        dX_out = [torch.empty_like(X) for _ in range(2)]                                    # remote, home
        Xb[0].copy_(X)
        tb[0].copy_(t)
        Lb[0][0].copy_(lse)
        Lb[0][1].copy_(dloss)
        acc_moving = None
        for i in range(P):
            owner = (r - i) % P
            c, n = i % 2, (i + 1) % 2
            ops_moving = self.tp.exchange([Xb[c], tb[c], Lb[c]], [Xb[n], tb[n], Lb[n]]) if i < P - 1 else None
            M.backward_meeting(Xb[c], W_own, tb[c], Lb[c][0], Lb[c][1], lo, self.V, self.ignore_index, _b.PHASE_RESIDUAL,
                               None, i == 0, i == P - 1, None, None, False, ws)
            if acc_moving is not None:
                acc_moving.wait()                         # this batch's dX accumulator, from rank r-1
            M.backward_meeting(Xb[c], W_own, tb[c], Lb[c][0], Lb[c][1], lo, self.V, self.ignore_index,
                               _b.PHASE_INPUT_GRAD, Ab[c], i == 0, i == P - 1, dX_out[0], None, False, ws)
            acc_moving = self.tp.exchange([Ab[c]], [Ab[n]]) if i < P - 1 else None   # the gradient travels with X
            M.backward_meeting(Xb[c], W_own, tb[c], Lb[c][0], Lb[c][1], lo, self.V, self.ignore_index,
                               _b.PHASE_WEIGHT_GRAD, None, i == 0, i == P - 1, None, dW_own, accumulate_dW or i > 0, ws)
            self._note("bwd", i, owner, r)
            if ops_moving is not None:
                ops_moving.wait()
        self.tp.exchange([dX_out[0]], [dX_out[1]]).wait()     # the finished dX goes home
        return dX_out[1], dW_own
