"""Seeded synthetic inputs for the fused vocabulary-projection + cross-entropy path.

This module is the only code shared by the CUDA path's callers (tests, bench) and the
float64 oracle.  It holds no arithmetic of the method itself: it draws random hidden
states, projection weights and target ids, rounds the floating-point draws to bfloat16
(round-to-nearest-even on the bit pattern) and hands out the *same* bit patterns to both
sides.  The shapes, value scales and label mix are those of the five benchmark workloads;
they stand in for the paper's MoE training workloads (its isolated benchmark, App. C, uses
random hidden states with H=7168 and V=200000 and describes no targets).

Recipe
------
* one ``numpy.random.Generator(PCG64)`` per array (labels, masks) or per slab of 4096 rows
  (H, W), seeded by ``SeedSequence([seed, stream_id, call_index(, slab)])`` (stream ids below),
  so arrays are independent, slabs can be drawn by several threads with the same result, and
  any call of a streamed workload can be regenerated alone;
* H ~ N(0, 1), W ~ N(0, w_std^2): float32 normals scaled in float32, then rounded to bf16;
* labels: uniform over [0, V) or truncated Zipf(s) over ranks 1..V with id = rank-1,
  sampled by inverse CDF (float64 ``searchsorted``);
* ignored positions: the first ``round(ignore_frac * T_stream)`` entries of a seeded
  permutation of the whole token stream get ``ignore_index``.
"""
from __future__ import annotations

import dataclasses
import hashlib
import os
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Optional

import numpy as np

STREAM_H = 1
STREAM_W = 2
STREAM_LABELS = 3
STREAM_IGNORE = 4
STREAM_DLOSS = 5

IGNORE_INDEX = -100


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and distribution of one benchmark workload.

    ``T`` is the number of tokens of ONE library call; ``n_calls`` such calls make the
    token stream (only the long-context workload has more than one).  ``T_chunk`` is the
    internal token chunk (the paper's per-rank batch N), ``block_v`` the vocabulary shard
    width (the paper's V/P).
    """

    name: str
    T: int
    d: int
    V: int
    block_v: int
    T_chunk: int
    w_std: float
    labels: str            # "uniform" | "zipf"
    zipf_s: float
    ignore_frac: float
    seed: int
    n_calls: int = 1

    @property
    def P(self) -> int:
        return -(-self.V // self.block_v)

    @property
    def T_stream(self) -> int:
        return self.T * self.n_calls

    @property
    def n_ignored(self) -> int:
        return int(round(self.ignore_frac * self.T_stream))

    @property
    def flops(self) -> float:
        """Algorithmic work of forward + recompute + both gradient contractions."""
        return 8.0 * self.T_stream * self.V * self.d

    @property
    def logits_bytes_fp32(self) -> int:
        return 4 * self.T_stream * self.V


WORKLOADS: Dict[str, Workload] = {
    w.name: w
    for w in [
        Workload("tiny", T=512, d=256, V=4096, block_v=512, T_chunk=128,
                 w_std=1.0 / 16.0, labels="uniform", zipf_s=0.0, ignore_frac=0.0, seed=0),
        Workload("mid", T=4096, d=2048, V=32768, block_v=4096, T_chunk=2048,
                 w_std=0.02, labels="zipf", zipf_s=1.1, ignore_frac=0.10, seed=1),
        Workload("moe120b", T=16384, d=2880, V=201088, block_v=8192, T_chunk=4096,
                 w_std=0.02, labels="zipf", zipf_s=1.1, ignore_frac=0.05, seed=2),
        Workload("moe667b", T=65536, d=7168, V=129280, block_v=8192, T_chunk=8192,
                 w_std=0.006, labels="zipf", zipf_s=1.1, ignore_frac=0.02, seed=3),
        Workload("longctx", T=16384, d=2880, V=201088, block_v=8192, T_chunk=4096,
                 w_std=0.02, labels="zipf", zipf_s=1.1, ignore_frac=0.01, seed=4, n_calls=64),
    ]
}


# Reduced cases of the moe120b / moe667b shapes for profiler captures: operands larger than the
# 126 MB L2 but well under a gigabyte on the device, a few launches per kernel kind.
PROFILE_WORKLOADS: Dict[str, Workload] = {
    w.name: w
    for w in [
        Workload("prof120b", T=4096, d=2880, V=32768, block_v=8192, T_chunk=4096,
                 w_std=0.02, labels="zipf", zipf_s=1.1, ignore_frac=0.05, seed=12),
        Workload("prof667b", T=4096, d=7168, V=16384, block_v=8192, T_chunk=4096,
                 w_std=0.006, labels="zipf", zipf_s=1.1, ignore_frac=0.02, seed=13),
        # The shape of the paper's isolated Ring-DTP benchmark (App. C: N = 16384 tokens per GPU, H = 7168,
        # V = 200000, P = 8), for a context line beside its Table 2; V/P = 25000 is rounded up to the next
        # multiple of the 256-column tile.  The paper runs it in FP32, this build in bf16.
        Workload("papershape32k", T=32768, d=7168, V=200000, block_v=25088, T_chunk=32768,
                 w_std=0.006, labels="zipf", zipf_s=1.1, ignore_frac=0.0, seed=15),
        Workload("papershape", T=16384, d=7168, V=200000, block_v=25088, T_chunk=16384,
                 w_std=0.006, labels="zipf", zipf_s=1.1, ignore_frac=0.0, seed=14),
    ]
}


# --------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to float32 exactly."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to float64 exactly (row slabs in a thread pool when large)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if bits.ndim != 2 or bits.size < (1 << 24):
        return bf16_bits_to_f32(bits).astype(np.float64)
    out = np.empty(bits.shape, dtype=np.float64)
    step = max(1, (1 << 22) // bits.shape[1])

    def conv(r0: int) -> None:
        out[r0:r0 + step] = bf16_bits_to_f32(bits[r0:r0 + step])

    with ThreadPoolExecutor(max(1, min(16, os.cpu_count() or 1))) as ex:
        list(ex.map(conv, range(0, bits.shape[0], step)))
    return out


# --------------------------------------------------------------------------- generators
def _rng(seed: int, stream: int, call_index: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, stream, call_index])))


SLAB_ROWS = 4096       # part of the recipe: each slab of rows has its own generator


def _threads() -> int:
    return max(1, min(16, os.cpu_count() or 1))


def gaussian_bf16(shape, std: float, seed: int, stream: int, call_index: int = 0) -> np.ndarray:
    """N(0, std^2) draws rounded to bf16, returned as uint16 bit patterns of ``shape``.

    Slab k (rows [k*SLAB_ROWS, (k+1)*SLAB_ROWS)) is drawn from its own generator
    SeedSequence([seed, stream, call_index, k]); slabs are filled by a thread pool, and the
    result does not depend on the number of threads.
    """
    rows, cols = int(shape[0]), int(shape[1])
    out = np.empty((rows, cols), dtype=np.uint16)
    s = np.float32(std)

    def fill(k: int) -> None:
        r0, r1 = k * SLAB_ROWS, min(rows, (k + 1) * SLAB_ROWS)
        rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, stream, call_index, k])))
        x = rng.standard_normal((r1 - r0, cols), dtype=np.float32)
        if std != 1.0:
            x *= s
        out[r0:r1] = f32_to_bf16_bits(x)

    n_slabs = -(-rows // SLAB_ROWS)
    if n_slabs == 1:
        fill(0)
    else:
        with ThreadPoolExecutor(_threads()) as ex:
            list(ex.map(fill, range(n_slabs)))
    return out


def f32_round_to_tf32(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest value with a 10-bit mantissa (TF32), ties to even; result is float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + (np.uint32(0xFFF) + ((u >> np.uint32(13)) & np.uint32(1)))) & np.uint32(0xFFFFE000)
    return r.view(np.float32)


def gaussian_f32(shape, std: float, seed: int, stream: int, call_index: int = 0, tf32: bool = True) -> np.ndarray:
    """N(0, std^2) float32 draws, same slab/seed scheme as gaussian_bf16; inputs of the FP32 (TF32 tensor
    core) entry points.  With ``tf32`` (default) the draws are rounded to TF32-representable values, so that
    the tensor core's products are exact and the float64 oracle sees the very numbers the GPU multiplies
    (the counterpart of rounding the bf16 path's inputs to bf16)."""
    rows, cols = int(shape[0]), int(shape[1])
    out = np.empty((rows, cols), dtype=np.float32)
    s = np.float32(std)

    def fill(k: int) -> None:
        r0, r1 = k * SLAB_ROWS, min(rows, (k + 1) * SLAB_ROWS)
        rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, stream, call_index, k])))
        x = rng.standard_normal((r1 - r0, cols), dtype=np.float32)
        if std != 1.0:
            x *= s
        out[r0:r1] = f32_round_to_tf32(x) if tf32 else x

    n_slabs = -(-rows // SLAB_ROWS)
    if n_slabs == 1:
        fill(0)
    else:
        with ThreadPoolExecutor(_threads()) as ex:
            list(ex.map(fill, range(n_slabs)))
    return out


def make_weights_f32(w: Workload, tf32: bool = True) -> np.ndarray:
    return gaussian_f32((w.V, w.d), w.w_std, w.seed, STREAM_W, 0, tf32)


def make_hidden_f32(w: Workload, call_index: int = 0, tf32: bool = True) -> np.ndarray:
    return gaussian_f32((w.T, w.d), 1.0, w.seed, STREAM_H, call_index, tf32)


def zipf_cdf(V: int, s: float) -> np.ndarray:
    """CDF of the Zipf law truncated to ranks 1..V, p(k) proportional to k^-s (float64)."""
    p = np.arange(1, V + 1, dtype=np.float64) ** (-float(s))
    c = np.cumsum(p)
    c /= c[-1]
    return c


def stream_labels(w: Workload) -> np.ndarray:
    """Targets of the whole token stream (all calls), int32, with ignored positions set."""
    n = w.T_stream
    rng = _rng(w.seed, STREAM_LABELS, 0)
    if w.labels == "uniform":
        lab = rng.integers(0, w.V, size=n, dtype=np.int64)
    elif w.labels == "zipf":
        u = rng.random(n)
        lab = np.searchsorted(zipf_cdf(w.V, w.zipf_s), u, side="left")
        lab = np.minimum(lab, w.V - 1)
    else:
        raise ValueError(w.labels)
    lab = lab.astype(np.int32)
    k = w.n_ignored
    if k:
        perm = _rng(w.seed, STREAM_IGNORE, 0).permutation(n)
        lab[perm[:k]] = IGNORE_INDEX
    return lab


@dataclasses.dataclass
class Batch:
    """One call's inputs: bf16 bit patterns for H and W, int32 labels."""

    H_bits: np.ndarray      # [T, d] uint16
    W_bits: np.ndarray      # [V, d] uint16
    labels: np.ndarray      # [T] int32
    call_index: int
    workload: Workload

    def checksums(self) -> Dict[str, str]:
        return {k: hashlib.sha256(np.ascontiguousarray(v).tobytes()).hexdigest()
                for k, v in (("H", self.H_bits), ("W", self.W_bits), ("labels", self.labels))}


def make_weights(w: Workload) -> np.ndarray:
    return gaussian_bf16((w.V, w.d), w.w_std, w.seed, STREAM_W, 0)


def make_hidden(w: Workload, call_index: int = 0) -> np.ndarray:
    return gaussian_bf16((w.T, w.d), 1.0, w.seed, STREAM_H, call_index)


def make_batch(w: Workload, call_index: int = 0, W_bits: Optional[np.ndarray] = None,
               labels_stream: Optional[np.ndarray] = None) -> Batch:
    """Inputs of call ``call_index`` of workload ``w`` (weights are shared by all calls)."""
    if not 0 <= call_index < w.n_calls:
        raise ValueError("call_index out of range")
    if W_bits is None:
        W_bits = make_weights(w)
    if labels_stream is None:
        labels_stream = stream_labels(w)
    lab = labels_stream[call_index * w.T:(call_index + 1) * w.T].copy()
    return Batch(make_hidden(w, call_index), W_bits, lab, call_index, w)


def custom_workload(name: str, T: int, d: int, V: int, block_v: int, T_chunk: int,
                    w_std: float = 0.05, labels: str = "uniform", zipf_s: float = 1.1,
                    ignore_frac: float = 0.0, seed: int = 1234) -> Workload:
    """A workload of arbitrary shape for edge-case tests (ragged V, tiny T, sharp logits)."""
    return Workload(name, T=T, d=d, V=V, block_v=block_v, T_chunk=T_chunk, w_std=w_std,
                    labels=labels, zipf_s=zipf_s, ignore_frac=ignore_frac, seed=seed)


def make_dloss(w: Workload, call_index: int = 0) -> np.ndarray:
    """A per-token upstream gradient (float32, uniform in [0.5, 1.5) / T) for tests that
    exercise the explicit-dloss argument."""
    rng = _rng(w.seed, STREAM_DLOSS, call_index)
    return ((0.5 + rng.random(w.T)) / w.T).astype(np.float32)
