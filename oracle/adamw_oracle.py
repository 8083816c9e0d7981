"""Float64 CPU oracle for the bucket-streamed AdamW update (OffloadStreamAdamW).

TEST INFRASTRUCTURE ONLY.  Nothing in the product path imports this file: it is used by ``tests/`` and by the
benchmark's CPU-baseline leg.  It shares no code with the CUDA path.

What the method computes (paper section 3.4; appendix "OffloadStreamAdamW", Algorithm 4)
----------------------------------------------------------------------------------------
The optimizer state of a rank (fp32 master weights, first and second moments) and the final gradients live in
host memory; they are cut into buckets of at most beta parameters, and every bucket is updated by one fused
AdamW step that also refreshes the bf16 working weight.  The appendix states that the fused kernel applies the
same bias correction, weight decay and update order as decoupled weight decay AdamW, so the result has a plain
definition, written out in ``adamw_step``.  With g the gradient, t = 1, 2, ... the step count:

    p <- p (1 - lr * weight_decay)                       decoupled decay, applied first
    m <- beta1 m + (1 - beta1) g
    v <- beta2 v + (1 - beta2) g^2
    p <- p - lr * (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps)
    w  = bf16(p)                                         working weight, round to nearest even

``streamed_step`` restates Algorithm 4's bucket loop (one bucket at a time, in order) to show that bucketing
changes nothing: the update is elementwise.  The bf16 refresh rounds the NEW fp32 master value (the state that is
written back is fp32), so ``adamw_step`` returns the master rounded to float32 first and the working weight as the
bf16 rounding of that float32 value.

Readings taken where the paper is silent:
* the order "decay, moments, update" and the placement of eps outside the square root of the bias-corrected
  second moment follow Loshchilov & Hutter's AdamW as implemented by ``torch.optim.AdamW`` (the paper cites it as
  "the reference implementation");
* no gradient clipping or scaling is part of the fused update (the appendix places global clipping outside it);
* buckets of a flat parameter shard are contiguous ranges (the paper groups whole tensors, which is the same
  thing for an elementwise rule).

Pinned by tests/test_adamw_oracle_pins.py: a hand-worked step, closed forms (t = 1 gives lr * sign(g) up to eps;
lr = 0; g = 0), torch.optim.AdamW in float64 over several steps, and bucket invariance.
"""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import numpy as np


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def adamw_step(p: np.ndarray, m: np.ndarray, v: np.ndarray, g: np.ndarray, step: int, lr: float, beta1: float,
               beta2: float, eps: float, weight_decay: float) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """One AdamW step in float64 on float32 state.  Returns (p_new, m_new, v_new) as float64 arrays holding the
    exact float64 results, and the working weight as bf16 bit patterns of float32(p_new)."""
    if step < 1:
        raise ValueError("step counts from 1")
    p = np.asarray(p, dtype=np.float64)
    m = np.asarray(m, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    p = p * (1.0 - lr * weight_decay)
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    m_hat = m / (1.0 - beta1 ** step)
    v_hat = v / (1.0 - beta2 ** step)
    p = p - lr * m_hat / (np.sqrt(v_hat) + eps)
    w_bits = f32_to_bf16_bits(p.astype(np.float32))
    return p, m, v, w_bits


def bucket_ranges(n: int, bucket_params: int, offsets: Optional[Sequence[int]] = None):
    """Algorithm 4, first line: buckets g = 1..G of at most beta parameters, in parameter order."""
    if offsets is not None:
        offs = [int(o) for o in offsets]
        if offs[0] != 0 or offs[-1] != n or any(b <= a for a, b in zip(offs, offs[1:])):
            raise ValueError("bucket offsets must rise from 0 to n")
        return list(zip(offs[:-1], offs[1:]))
    if bucket_params < 1:
        raise ValueError("bucket size must be positive")
    return [(a, min(n, a + bucket_params)) for a in range(0, n, bucket_params)]


def streamed_step(p, m, v, g, step, lr, beta1, beta2, eps, weight_decay, bucket_params: int,
                  offsets: Optional[Sequence[int]] = None):
    """Algorithm 4: the same update, one bucket after the other (host state in, host state out)."""
    n = len(p)
    po, mo, vo = np.empty(n), np.empty(n), np.empty(n)
    wo = np.empty(n, dtype=np.uint16)
    for a, b in bucket_ranges(n, bucket_params, offsets):
        po[a:b], mo[a:b], vo[a:b], wo[a:b] = adamw_step(p[a:b], m[a:b], v[a:b], g[a:b], step, lr, beta1, beta2, eps,
                                                        weight_decay)
    return po, mo, vo, wo
