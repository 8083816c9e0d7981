"""Forward + backward for callers whose activations live in HOST memory, with the copies taken off the critical path.

``vp_ce_fwd_bwd_host`` (the C entry point) copies in, computes, copies out and synchronises: the link time (two times
``T * d * 2`` bytes) is added to every step.  A training loop does not have to pay it: the hidden states of step i+1
can travel to the device while step i computes, and the input gradient of step i can travel back while step i+1
computes.  ``HostStepPipeline`` does exactly that with ``depth`` sets of device staging buffers and two copy streams.
It holds no arithmetic: every step is ``vp_ce_forward`` + ``vp_ce_backward`` (masked-mean upstream gradient) on the
caller's stream; torch supplies streams, events and memory.

    pipe = HostStepPipeline(W, dW, T, d, block_v=8192, T_chunk=16384)
    for step in range(n):
        pipe.submit(H_host[step], labels_host[step], loss_host[step], dH_host[step])   # pinned CPU tensors; returns at once
    pipe.wait()                                                                       # all host outputs are valid now

Host outputs of a submitted step are valid after ``wait()`` (or after a later ``submit`` has reused the same slot:
``submit`` first waits, on the host, for the copy-out of the step that used the slot ``depth`` submits earlier).
"""
from __future__ import annotations

from typing import List, Optional

import torch

from . import binding as _b


class HostStepPipeline:
    def __init__(self, W: torch.Tensor, dW: torch.Tensor, T: int, d: int, block_v: int, T_chunk: int,
                 ignore_index: int = -100, depth: int = 2, accumulate_dW: bool = False):
        if depth < 1:
            raise ValueError("depth must be at least 1")
        dev = W.device
        self.W, self.dW = W, dW
        self.T, self.d, self.block_v, self.T_chunk = int(T), int(d), int(block_v), int(T_chunk)
        self.ignore_index, self.accumulate_dW = int(ignore_index), bool(accumulate_dW)
        self.depth = depth
        n = _b.vp_ce_workspace_bytes(self.T_chunk, self.d, self.block_v)
        if n == 0:
            raise ValueError("unsupported shape: d % 8, block_v % 256 or T_chunk % 128")
        self.ws = torch.empty(n, dtype=torch.uint8, device=dev)         # one workspace: steps compute one after the other
        self.H = [torch.empty(T, d, dtype=torch.bfloat16, device=dev) for _ in range(depth)]
        self.labels = [torch.empty(T, dtype=torch.int32, device=dev) for _ in range(depth)]
        self.loss = [torch.empty(T, dtype=torch.float32, device=dev) for _ in range(depth)]
        self.lse = [torch.empty(T, dtype=torch.float32, device=dev) for _ in range(depth)]
        self.dH = [torch.empty(T, d, dtype=torch.bfloat16, device=dev) for _ in range(depth)]
        self.s_in = torch.cuda.Stream(dev)
        self.s_out = torch.cuda.Stream(dev)
        self.ev_in: List[Optional[torch.cuda.Event]] = [None] * depth        # slot's inputs have arrived
        self.ev_done: List[Optional[torch.cuda.Event]] = [None] * depth      # slot's compute has finished
        self.ev_out: List[Optional[torch.cuda.Event]] = [None] * depth       # slot's outputs have left
        self.step = 0
        self.chunks_per_call = -(-self.T // self.T_chunk)

    def submit(self, H_host: torch.Tensor, labels_host: torch.Tensor, loss_host: torch.Tensor, dH_host: torch.Tensor,
               chunk_index_base: Optional[int] = None) -> None:
        """Enqueues one forward + backward step on host buffers (pinned memory makes the copies asynchronous)."""
        k = self.step % self.depth
        main = torch.cuda.current_stream(self.W.device)
        if self.ev_out[k] is not None:
            self.ev_out[k].synchronize()                     # the host buffers of the step that used this slot are complete,
        with torch.cuda.stream(self.s_in):                   # and its device buffers are free: copy the new inputs in
            self.H[k].copy_(H_host, non_blocking=True)
            self.labels[k].copy_(labels_host, non_blocking=True)
            self.ev_in[k] = torch.cuda.Event()
            self.ev_in[k].record(self.s_in)
        main.wait_event(self.ev_in[k])
        base = self.step * self.chunks_per_call if chunk_index_base is None else int(chunk_index_base)
        _b.vp_ce_forward(self.H[k], self.W, self.labels[k], self.block_v, self.ignore_index, self.loss[k], self.lse[k],
                         self.T_chunk, base, self.ws, stream=main)
        _b.vp_ce_backward(self.H[k], self.W, self.labels[k], self.lse[k], None, self.dH[k], self.dW, self.block_v,
                          self.ignore_index, self.T_chunk, base, self.accumulate_dW, self.ws, stream=main)
        self.ev_done[k] = torch.cuda.Event()
        self.ev_done[k].record(main)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_done[k])
            loss_host.copy_(self.loss[k], non_blocking=True)
            dH_host.copy_(self.dH[k], non_blocking=True)
            self.ev_out[k] = torch.cuda.Event()
            self.ev_out[k].record(self.s_out)
        self.step += 1

    def wait(self) -> None:
        """Blocks until the host outputs of every submitted step are complete."""
        for ev in self.ev_out:
            if ev is not None:
                ev.synchronize()

    def device_status(self) -> int:
        """Status word of the last backward (see vp_ce_device_status)."""
        return _b.vp_ce_device_status(self.ws)
