"""Float64 CPU oracle for the vocabulary projection fused with cross-entropy.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path imports this file: it is used by
``tests/``, by the smoke check and by the benchmark's CPU-baseline leg.  It shares no code
with the CUDA path.  It is slow and plain on purpose so that it can be checked against the
paper by eye.

What the method computes (paper §3.2, Eq. 2, App. C / Algorithm 3)
------------------------------------------------------------------
The method visits the vocabulary one shard at a time and keeps, per token, only the running
state S = (m, z, y_t); after all shards the negative log-likelihood is m + log z - y_t
(§3.2, sentence after Eq. 2; Algorithm 3 output line).  The paper states that only order
and granularity change and that loss and gradients stay exact, so the reference result has
a plain definition, which is what the ``dense_*`` functions write out:

    y[n, v]  = sum_k H[n, k] * W[v, k]
    lse[n]   = max_v y[n, v] + log sum_v exp(y[n, v] - max_v y[n, v])
    loss[n]  = lse[n] - y[n, t_n]        (0 when t_n == ignore_index)
    G[n, v]  = dloss[n] * (exp(y[n, v] - lse[n]) - [v == t_n])      (row 0 when ignored)
    dH[n, :] = sum_v G[n, v] * W[v, :]          dW[v, :] = sum_n G[n, v] * H[n, :]

The backward formulas are the textbook softmax cross-entropy gradient; App. C describes
them in prose only ("forms the softmax residual for one strip at a time, and contracts it
into input and weight gradients").

``ring_fold_forward`` / ``ring_backward`` restate Algorithm 3 step by step (Fold with the
initial state (-inf, 0, 0), shards met in the order q = (r - i) mod P) in float64, to check
Eq. 2 and the rotation against the dense definition.

Readings taken where the paper is silent (each is also listed in the design notes):
* the weight is stored [V, d] row-major and logits are H @ W.T (the paper writes W as
  H x V, column-sharded: same mathematics);
* a token whose target equals ``ignore_index`` has loss 0, a zero residual row and is
  excluded from n_valid; its lse is still returned;
* ``dloss=None`` means the masked mean: 1/n_valid for valid tokens; n_valid == 0 gives
  mean 0 and zero gradients;
* a target outside [0, V) other than ``ignore_index`` is an error here (ValueError);
* on one device the ring rank r becomes the global token-chunk index.

Every function here is pinned by tests/test_oracle_pins.py (closed forms, finite
differences, brute-force loops, library special cases); none is "parity unpinned".
"""
from __future__ import annotations

import math
from typing import Optional, Sequence, Tuple

import numpy as np


# ----------------------------------------------------------------------------- helpers
def _check_labels(labels: np.ndarray, V: int, ignore_index: int) -> np.ndarray:
    labels = np.asarray(labels).astype(np.int64)
    valid = labels != ignore_index
    bad = valid & ((labels < 0) | (labels >= V))
    if bad.any():
        raise ValueError("label outside [0, V) that is not ignore_index")
    return valid


def default_dloss(labels: np.ndarray, ignore_index: int) -> np.ndarray:
    """Upstream gradient of the masked-mean loss: 1/n_valid on valid tokens, else 0."""
    valid = np.asarray(labels) != ignore_index
    n_valid = int(valid.sum())
    out = np.zeros(valid.shape[0], dtype=np.float64)
    if n_valid:
        out[valid] = 1.0 / n_valid
    return out


def masked_mean(loss: np.ndarray, labels: np.ndarray, ignore_index: int) -> Tuple[float, int]:
    """Mean of per-token loss over valid tokens; (0.0, 0) when there is none."""
    valid = np.asarray(labels) != ignore_index
    n_valid = int(valid.sum())
    if n_valid == 0:
        return 0.0, 0
    return float(np.asarray(loss, dtype=np.float64)[valid].sum() / n_valid), n_valid


# ----------------------------------------------------------------------------- dense definition
def dense_forward(H: np.ndarray, W: np.ndarray, labels: np.ndarray, ignore_index: int = -100,
                  slab: int = 1024) -> Tuple[np.ndarray, np.ndarray]:
    """Per-token (lse, loss) from fully materialised logits, one slab of tokens at a time.

    §3.2: NLL = m + log z - y_t, with m the row maximum and z the sum of exp(y - m); this is
    the plain log-sum-exp.  H [T, d], W [V, d] are float64 (bf16 values widened exactly).
    """
    H = np.asarray(H, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    T, V = H.shape[0], W.shape[0]
    valid = _check_labels(labels, V, ignore_index)
    lab = np.asarray(labels).astype(np.int64)
    lse = np.empty(T, dtype=np.float64)
    loss = np.zeros(T, dtype=np.float64)
    for n0 in range(0, T, slab):
        n1 = min(T, n0 + slab)
        y = H[n0:n1] @ W.T                                   # [slab, V] logits
        m = y.max(axis=1)
        z = np.exp(y - m[:, None]).sum(axis=1)
        lse[n0:n1] = m + np.log(z)
        rows = np.nonzero(valid[n0:n1])[0]
        loss[n0 + rows] = lse[n0 + rows] - y[rows, lab[n0 + rows]]
    return lse, loss


def dense_backward(H: np.ndarray, W: np.ndarray, labels: np.ndarray,
                   dloss: Optional[np.ndarray] = None, ignore_index: int = -100,
                   slab: int = 1024) -> Tuple[np.ndarray, np.ndarray]:
    """(dH [T, d], dW [V, d]) from the materialised softmax residual G (App. C prose)."""
    H = np.asarray(H, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    T, V = H.shape[0], W.shape[0]
    valid = _check_labels(labels, V, ignore_index)
    lab = np.asarray(labels).astype(np.int64)
    dl = default_dloss(labels, ignore_index) if dloss is None else np.asarray(dloss, dtype=np.float64)
    dH = np.zeros_like(H)
    dW = np.zeros_like(W)
    for n0 in range(0, T, slab):
        n1 = min(T, n0 + slab)
        y = H[n0:n1] @ W.T
        m = y.max(axis=1, keepdims=True)
        lse = m + np.log(np.exp(y - m).sum(axis=1, keepdims=True))
        G = np.exp(y - lse)                                   # softmax
        rows = np.nonzero(valid[n0:n1])[0]
        G[rows, lab[n0 + rows]] -= 1.0                        # minus one-hot
        G *= dl[n0:n1, None]
        G[~valid[n0:n1]] = 0.0                                # ignored tokens contribute nothing
        dH[n0:n1] = G @ W
        dW += G.T @ H[n0:n1]
    return dH, dW


def naive_forward_backward(H, W, labels, dloss=None, ignore_index=-100):
    """The same definition in pure Python loops (tiny inputs only); no library contraction."""
    T, d = len(H), len(H[0])
    V = len(W)
    n_valid = sum(1 for t in labels if t != ignore_index)
    lse = [0.0] * T
    loss = [0.0] * T
    dH = [[0.0] * d for _ in range(T)]
    dW = [[0.0] * d for _ in range(V)]
    for n in range(T):
        y = [sum(float(H[n][k]) * float(W[v][k]) for k in range(d)) for v in range(V)]
        m = max(y)
        z = sum(math.exp(yv - m) for yv in y)
        lse[n] = m + math.log(z)
        t = int(labels[n])
        if t == ignore_index:
            continue
        if not 0 <= t < V:
            raise ValueError("label outside [0, V)")
        loss[n] = lse[n] - y[t]
        g_up = (1.0 / n_valid) if dloss is None else float(dloss[n])
        for v in range(V):
            g = g_up * (math.exp(y[v] - lse[n]) - (1.0 if v == t else 0.0))
            for k in range(d):
                dH[n][k] += g * float(W[v][k])
                dW[v][k] += g * float(H[n][k])
    return lse, loss, dH, dW


# ----------------------------------------------------------------------------- Algorithm 3
def fold(state: Tuple[np.ndarray, np.ndarray, np.ndarray], Y: np.ndarray, targets: np.ndarray,
         v_lo: int, v_hi: int):
    """Fold of Algorithm 3: update (m, z, y) of every token with one logit strip.

    Eq. 2: m' = max(m, max_v Y), z' = exp(m - m') z + sum_v exp(Y - m');
    if the target lies in the strip's interval [v_lo, v_hi) then y <- Y[n, t_n].
    Returns the new state and the mask of tokens whose target was gathered by this strip.
    """
    m, z, y = state
    m_new = np.maximum(m, Y.max(axis=1))
    with np.errstate(invalid="ignore"):
        scale = np.where(np.isneginf(m), 0.0, np.exp(m - m_new))   # exp(-inf - m') = 0, never inf - inf
    z_new = scale * z + np.exp(Y - m_new[:, None]).sum(axis=1)
    t = np.asarray(targets).astype(np.int64)
    own = (t >= v_lo) & (t < v_hi)
    y_new = y.copy()
    rows = np.nonzero(own)[0]
    y_new[rows] = Y[rows, t[rows] - v_lo]
    return (m_new, z_new, y_new), own


def shard_order(c: int, P: int, direction: int = -1, start_offset: int = 0) -> Sequence[int]:
    """Shards met by ring rank / global token chunk ``c``: q_i = (c - i) mod P, i = 0..P-1
    (Algorithm 3's first Fold uses the rank's own shard, i = 0).  ``direction=+1`` and
    ``start_offset`` exist only to test order invariance."""
    return [int((c + start_offset + direction * i) % P) for i in range(P)]


def ring_fold_forward(H: np.ndarray, W: np.ndarray, labels: np.ndarray, block_v: int,
                      T_chunk: int, chunk_index_base: int = 0, ignore_index: int = -100,
                      direction: int = -1, start_offset: int = 0):
    """Algorithm 3 on one device: token chunks play the ranks, shards of ``block_v`` rows of
    W are met in rotated order, each meeting forms one strip, folds it and drops it.

    Returns (lse, loss, gathers) where gathers[n] counts how many meetings supplied y_t for
    token n (App. C: exactly one for a valid target)."""
    H = np.asarray(H, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    T, V = H.shape[0], W.shape[0]
    valid = _check_labels(labels, V, ignore_index)
    lab = np.asarray(labels).astype(np.int64)
    P = -(-V // block_v)
    lse = np.empty(T, dtype=np.float64)
    loss = np.zeros(T, dtype=np.float64)
    gathers = np.zeros(T, dtype=np.int64)
    n_chunks = -(-T // T_chunk)
    for c in range(n_chunks):
        n0, n1 = c * T_chunk, min(T, (c + 1) * T_chunk)
        X, t = H[n0:n1], lab[n0:n1]
        S = (np.full(n1 - n0, -np.inf), np.zeros(n1 - n0), np.zeros(n1 - n0))   # (-inf, 0, 0)
        for q in shard_order(chunk_index_base + c, P, direction, start_offset):
            v_lo, v_hi = q * block_v, min(V, (q + 1) * block_v)
            Y = X @ W[v_lo:v_hi].T                         # the strip; released after the fold
            t_in = np.where(valid[n0:n1], t, -1)           # ignored tokens own no column
            S, own = fold(S, Y, t_in, v_lo, v_hi)
            gathers[n0:n1] += own.astype(np.int64)
        m, z, y = S
        lse[n0:n1] = m + np.log(z)
        nll = m + np.log(z) - y                            # Algorithm 3 output line
        loss[n0:n1] = np.where(valid[n0:n1], nll, 0.0)
    return lse, loss, gathers


def ring_backward(H: np.ndarray, W: np.ndarray, labels: np.ndarray, lse: np.ndarray,
                  block_v: int, T_chunk: int, chunk_index_base: int = 0,
                  dloss: Optional[np.ndarray] = None, ignore_index: int = -100):
    """Backward as App. C describes it: replay the meetings, recompute one strip at a time,
    form its residual from the saved normaliser and contract it into dH and dW."""
    H = np.asarray(H, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    T, V = H.shape[0], W.shape[0]
    valid = _check_labels(labels, V, ignore_index)
    lab = np.asarray(labels).astype(np.int64)
    dl = default_dloss(labels, ignore_index) if dloss is None else np.asarray(dloss, dtype=np.float64)
    dl = np.where(valid, dl, 0.0)
    P = -(-V // block_v)
    dH = np.zeros_like(H)
    dW = np.zeros_like(W)
    for c in range(-(-T // T_chunk)):
        n0, n1 = c * T_chunk, min(T, (c + 1) * T_chunk)
        X = H[n0:n1]
        for q in shard_order(chunk_index_base + c, P):
            v_lo, v_hi = q * block_v, min(V, (q + 1) * block_v)
            Y = X @ W[v_lo:v_hi].T
            G = np.exp(Y - np.asarray(lse, dtype=np.float64)[n0:n1, None])
            own = valid[n0:n1] & (lab[n0:n1] >= v_lo) & (lab[n0:n1] < v_hi)
            rows = np.nonzero(own)[0]
            G[rows, lab[n0 + rows] - v_lo] -= 1.0
            G *= dl[n0:n1, None]
            dH[n0:n1] += G @ W[v_lo:v_hi]
            dW[v_lo:v_hi] += G.T @ X
    return dH, dW


# ----------------------------------------------------------------------------- sampled outputs
def rows_forward(H_rows: np.ndarray, W: np.ndarray, labels_rows: np.ndarray,
                 ignore_index: int = -100, v_slab: int = 32768):
    """(lse, loss) of a few tokens against the whole vocabulary, W taken slab by slab so that
    W may be handed over as a callable ``W(v0, v1) -> float64 [v1-v0, d]`` or an array."""
    H_rows = np.asarray(H_rows, dtype=np.float64)
    getW, V = _w_getter(W)
    lab = np.asarray(labels_rows).astype(np.int64)
    valid = lab != ignore_index
    if (valid & ((lab < 0) | (lab >= V))).any():
        raise ValueError("label outside [0, V)")
    ys = [H_rows @ getW(v0, min(V, v0 + v_slab)).T for v0 in range(0, V, v_slab)]
    y = np.concatenate(ys, axis=1)
    m = y.max(axis=1)
    lse = m + np.log(np.exp(y - m[:, None]).sum(axis=1))
    loss = np.zeros_like(lse)
    r = np.nonzero(valid)[0]
    loss[r] = lse[r] - y[r, lab[r]]
    return lse, loss, y


def rows_dH(H_rows: np.ndarray, W, labels_rows: np.ndarray, dloss_rows: np.ndarray,
            ignore_index: int = -100, v_slab: int = 32768) -> np.ndarray:
    """dH rows of a few tokens: dloss_n (sum_v p_v W_v - W_{t_n})."""
    lse, _, y = rows_forward(H_rows, W, labels_rows, ignore_index, v_slab)
    getW, V = _w_getter(W)
    lab = np.asarray(labels_rows).astype(np.int64)
    valid = lab != ignore_index
    G = np.exp(y - lse[:, None])
    r = np.nonzero(valid)[0]
    G[r, lab[r]] -= 1.0
    G *= np.where(valid, np.asarray(dloss_rows, dtype=np.float64), 0.0)[:, None]
    out = np.zeros_like(np.asarray(H_rows, dtype=np.float64))
    for v0 in range(0, V, v_slab):
        v1 = min(V, v0 + v_slab)
        out += G[:, v0:v1] @ getW(v0, v1)
    return out


def rows_dW(v_idx: np.ndarray, H: np.ndarray, W_rows: np.ndarray, labels: np.ndarray,
            lse: np.ndarray, dloss: np.ndarray, ignore_index: int = -100) -> np.ndarray:
    """dW rows of a few vocabulary ids, given the oracle's lse of EVERY token:
    dW[v, :] = sum_n dloss_n (exp(H_n . W_v - lse_n) - [t_n == v]) H_n."""
    H = np.asarray(H, dtype=np.float64)
    W_rows = np.asarray(W_rows, dtype=np.float64)
    lab = np.asarray(labels).astype(np.int64)
    valid = lab != ignore_index
    dl = np.where(valid, np.asarray(dloss, dtype=np.float64), 0.0)
    y = H @ W_rows.T                                        # [T, k]
    G = np.exp(y - np.asarray(lse, dtype=np.float64)[:, None])
    for j, v in enumerate(np.asarray(v_idx).astype(np.int64)):
        G[valid & (lab == v), j] -= 1.0
    G *= dl[:, None]
    return G.T @ H


def _w_getter(W):
    if callable(W):
        raise TypeError("pass (callable, V) as a tuple")
    if isinstance(W, tuple):
        return W[0], int(W[1])
    W = np.asarray(W, dtype=np.float64)
    return (lambda a, b: W[a:b]), W.shape[0]


# ----------------------------------------------------------------------------- whole pass (timed CPU baseline)
def forward_backward(H: np.ndarray, W: np.ndarray, labels: np.ndarray,
                     dloss: Optional[np.ndarray] = None, ignore_index: int = -100, slab: int = 1024):
    """Forward + backward by the dense definition; what the benchmark's CPU leg times."""
    lse, loss = dense_forward(H, W, labels, ignore_index, slab)
    dH, dW = dense_backward(H, W, labels, dloss, ignore_index, slab)
    mean, n_valid = masked_mean(loss, labels, ignore_index)
    return dict(lse=lse, loss=loss, mean=mean, n_valid=n_valid, dH=dH, dW=dW)
