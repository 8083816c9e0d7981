"""torch.autograd front end of the fused vocabulary projection + cross-entropy.

``vocab_proj_cross_entropy(H, W, labels)`` returns the per-token negative log-likelihood (the output of
Algorithm 3) and is differentiable in ``H`` and ``W``: the backward pass is ``vp_ce_backward`` with the
incoming gradient as the per-token upstream gradient.  Argument marshalling only; every step of the path
runs in the CUDA library.  The tokens x vocabulary logits are never materialised, so peak memory is the
workspace, ``O(T_chunk * block_v)``, whatever V is.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as _b


def _pick_chunk(T: int, T_chunk: Optional[int]) -> int:
    if T_chunk is None:
        T_chunk = 16384
    T_chunk = min(int(T_chunk), -(-T // 128) * 128)
    return max(128, (T_chunk // 128) * 128)


class _VocabProjCE(torch.autograd.Function):
    @staticmethod
    def forward(ctx, H, W, labels, block_v, ignore_index, T_chunk, chunk_index_base, dW_accum):
        if H.dtype != torch.bfloat16 or W.dtype != torch.bfloat16:
            raise TypeError("H and W must be bfloat16 CUDA tensors")
        H = H.contiguous()
        W = W.contiguous()
        labels = labels.to(torch.int32).contiguous()
        T, d = H.shape
        T_chunk = _pick_chunk(T, T_chunk)
        ws = _workspace(T_chunk, d, block_v, H.device)
        loss = torch.empty(T, dtype=torch.float32, device=H.device)
        lse = torch.empty(T, dtype=torch.float32, device=H.device)
        _b.vp_ce_forward(H, W, labels, block_v, ignore_index, loss, lse, T_chunk, chunk_index_base, ws)
        ctx.save_for_backward(H, W, labels, lse)
        ctx.cfg = (block_v, ignore_index, T_chunk, chunk_index_base)
        ctx.dW_accum = dW_accum
        return loss

    @staticmethod
    def backward(ctx, grad_loss):
        H, W, labels, lse = ctx.saved_tensors
        block_v, ignore_index, T_chunk, base = ctx.cfg
        accum = ctx.dW_accum
        need_dH = ctx.needs_input_grad[0]
        need_dW = accum is not None or ctx.needs_input_grad[1]
        if not (need_dH or need_dW):
            return (None,) * 8
        # the workspace holds nothing between calls: it is taken from the caching allocator here, not kept alive
        # from forward to backward
        ws = _workspace(T_chunk, H.shape[1], block_v, H.device)
        dH = torch.empty_like(H) if need_dH else None
        dW = None
        if need_dW:
            dW = accum if accum is not None else torch.empty(W.shape, dtype=torch.float32, device=W.device)
        _b.vp_ce_backward(H, W, labels, lse, grad_loss.to(torch.float32).contiguous(), dH, dW, block_v, ignore_index,
                          T_chunk, base, accum is not None, ws)
        # with an fp32 accumulation buffer the weight gradient lives there (main-grad style); autograd gets none
        grad_W = None if (accum is not None or dW is None) else dW.to(W.dtype)
        return dH, grad_W, None, None, None, None, None, None


def _workspace(T_chunk: int, d: int, block_v: int, device) -> torch.Tensor:
    n = _b.vp_ce_workspace_bytes(T_chunk, d, block_v)
    if n == 0:
        raise ValueError("unsupported shape: d % 8, block_v % 256 or T_chunk % 128")
    return torch.empty(n, dtype=torch.uint8, device=device)


def vocab_proj_cross_entropy(H: torch.Tensor, W: torch.Tensor, labels: torch.Tensor, block_v: int = 8192,
                             ignore_index: int = -100, T_chunk: Optional[int] = None, chunk_index_base: int = 0,
                             dW_accum: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Per-token loss ``lse(H @ W.T) - (H @ W.T)[n, labels[n]]`` (0 for ignored tokens), float32 ``[T]``.

    H ``[T, d]`` and W ``[V, d]`` are bfloat16 CUDA tensors, ``labels`` ``[T]`` integer.  ``block_v`` is the
    vocabulary shard width (multiple of 256), ``T_chunk`` the token chunk (multiple of 128).  If ``dW_accum``
    (float32 ``[V, d]``) is given, the weight gradient is ADDED into it in fp32 and ``W.grad`` stays untouched;
    otherwise autograd receives it rounded to W's dtype.
    """
    return _VocabProjCE.apply(H, W, labels, int(block_v), int(ignore_index), T_chunk, int(chunk_index_base), dW_accum)


class _MaskedMean(torch.autograd.Function):
    """Masked mean of the per-token loss (vp_ce_mean_loss); its gradient is 1/n_valid on valid tokens."""

    @staticmethod
    def forward(ctx, loss, labels, V, ignore_index):
        labels = labels.to(torch.int32).contiguous()
        mean = torch.empty(1, dtype=torch.float32, device=loss.device)
        n_valid = torch.empty(1, dtype=torch.int32, device=loss.device)
        _b.vp_ce_mean_loss(loss.contiguous(), labels, V, ignore_index, mean, n_valid)
        ctx.save_for_backward(labels, n_valid)
        ctx.ignore_index, ctx.V = ignore_index, V
        return mean[0]

    @staticmethod
    def backward(ctx, g):
        labels, n_valid = ctx.saved_tensors
        dloss = torch.empty(labels.numel(), dtype=torch.float32, device=labels.device)
        _b.vp_ce_mean_loss_grad(labels, ctx.V, ctx.ignore_index, n_valid, g.to(torch.float32).reshape(1).contiguous(),
                                dloss)
        return dloss, None, None, None


def vocab_proj_cross_entropy_mean(H: torch.Tensor, W: torch.Tensor, labels: torch.Tensor, **kwargs) -> torch.Tensor:
    """Scalar masked-mean loss over tokens whose label is not ``ignore_index`` (0 when there is none);
    keyword arguments as for ``vocab_proj_cross_entropy``."""
    loss = vocab_proj_cross_entropy(H, W, labels, **kwargs)
    return _MaskedMean.apply(loss, labels, int(W.shape[0]), int(kwargs.get("ignore_index", -100)))
