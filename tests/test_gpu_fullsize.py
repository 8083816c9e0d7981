"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

The float64 oracle cannot materialise these problems in test time, so outputs are sampled:
* lse / loss / dH rows of sampled tokens are computed by the oracle one token at a time
  (a token's row needs only its own hidden state and the whole weight);
* dW under the benchmark's own DENSE upstream gradient (config 3): the oracle computes lse of every token once
  and then forms sampled rows of dW exactly (a row of dW needs every token but only its own row of W) -- the
  sample holds id 0 (the most frequent target), ids of the ragged last shard, targeted ids and ids that are no
  token's target (pure softmax part: no one-hot term whose rounding could mask a wrong softmax);
* dW with a sparse upstream gradient (all configs): dloss is non-zero on a token set that has one token in
  every 64-token k-block of the weight-gradient GEMM plus one whole 128-token tile, so dW = sum over those
  tokens and the oracle can form ALL of it, while the GPU still runs the full-size launches;
* invariants that hold at any size: column sums of dW vanish (each residual row sums to 0), every
  lse is finite, the workspace size does not depend on V or on the number of calls.
"""
import numpy as np
import pytest
import torch

import paper_2609_14306_b200 as vp
from bench import BENCH_T_CHUNK
from oracle import vpce_oracle as orc
from synth_inputs import (IGNORE_INDEX, WORKLOADS, bf16_bits_to_f64, make_hidden, make_weights,
                          stream_labels)
from vpce_testlib import TOL_GRAD, TOL_TOKEN, DeviceRun, relF, untargeted_ids

pytestmark = pytest.mark.gpu

_cache = {}


def weights(name):
    """Host bits, float64 copy and device copy of a workload's weight (shared by the tests below)."""
    key = (WORKLOADS[name].V, WORKLOADS[name].d, WORKLOADS[name].seed)
    if key not in _cache:
        _cache.clear()
        bits = make_weights(WORKLOADS[name])
        _cache[key] = (bits, bf16_bits_to_f64(bits))
    return _cache[key]


def sampled_tokens(T, per_tile=2, seed=0):
    rng = np.random.default_rng(seed)
    tiles = T // 128
    idx = (np.arange(tiles)[:, None] * 128 + rng.integers(0, 128, size=(tiles, per_tile))).ravel()
    return np.unique(np.concatenate([idx, [0, T - 1]]))


def sparse_token_set(T, seed):
    """One token in every 64-token block (each k-block of the weight-gradient GEMM then carries data) plus every
    token of one 128-token tile (every row position of a tile)."""
    rng = np.random.default_rng(seed)
    per_block = np.arange(T // 64) * 64 + rng.integers(0, 64, size=T // 64)
    tile = int(rng.integers(0, T // 128))
    return np.unique(np.concatenate([per_block, np.arange(tile * 128, (tile + 1) * 128), [0, T - 1]]))


def sampled_vocab_ids(labels, V, block_v, n, seed):
    """Vocabulary ids for the dense-dloss dW check: id 0, the first and last id of the (ragged) last shard, the
    most frequent targets, random targeted ids and random ids that are no token's target."""
    rng = np.random.default_rng(seed)
    never = untargeted_ids(labels, V)
    lab = labels[labels != IGNORE_INDEX]
    targeted = np.unique(lab)
    last0 = (V - 1) // block_v * block_v
    picks = [np.array([0, 1, last0, V - 1]),
             rng.choice(targeted, size=min(n // 4, len(targeted)), replace=False),
             rng.choice(never, size=min(n // 2, len(never)), replace=False),
             rng.integers(last0, V, size=n // 8),
             rng.integers(0, V, size=n // 8)]
    return np.unique(np.concatenate(picks)), never


def check_call(w, call, W_bits, W64, labels_stream, n_valid_total, T_chunk, W_dev=None, n_sample_tiles=None,
               dense_dW_rows=0):
    H_bits = make_hidden(w, call)
    labels = labels_stream[call * w.T:(call + 1) * w.T]
    base = call * (-(-w.T // T_chunk))
    run = DeviceRun(H_bits, W_bits, labels, w.block_v, T_chunk, base, W_dev=W_dev)
    run.forward()
    assert run.fwd_status == 0
    # ---- default (masked-mean over the stream) upstream gradient: lse, loss, dH on sampled tokens
    dl_full = np.where(labels != IGNORE_INDEX, 1.0 / n_valid_total, 0.0)
    run.backward(dloss=dl_full.astype(np.float32))
    assert run.bwd_status == 0
    rows = sampled_tokens(w.T, per_tile=1 if w.T > 20000 else 2, seed=call)
    if n_sample_tiles:
        rows = rows[:: max(1, len(rows) // n_sample_tiles)]
    H64_rows = bf16_bits_to_f64(H_bits[rows])
    lse_ref, loss_ref, _ = orc.rows_forward(H64_rows, W64, labels[rows], IGNORE_INDEX)
    lse, loss = run.np_lse(), run.np_loss()
    assert np.isfinite(lse).all() and np.isfinite(loss).all()
    assert np.abs(lse[rows] - lse_ref).max() <= TOL_TOKEN
    assert np.abs(loss[rows] - loss_ref).max() <= TOL_TOKEN
    assert not loss[labels == IGNORE_INDEX].any()
    dl32 = dl_full.astype(np.float32).astype(np.float64)
    dH_ref = orc.rows_dH(H64_rows, W64, labels[rows], dl32[rows], IGNORE_INDEX)
    dH_rows = run.dH[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    assert relF(dH_rows, dH_ref) <= TOL_GRAD
    assert not run.dH[torch.from_numpy(np.nonzero(labels == IGNORE_INDEX)[0]).cuda()].any()
    # invariant: every residual row sums to zero, so the column sums of dW vanish (up to bf16 rounding of G)
    colsum = run.dW.double().sum(0)
    assert float(colsum.norm() / run.dW.double().norm()) < 5e-4
    mean_gpu, n_valid = run.mean()
    valid = labels != IGNORE_INDEX
    assert n_valid == int(valid.sum())
    assert abs(mean_gpu - loss[valid].mean()) <= 1e-4 * abs(loss[valid].mean())
    # ---- the same dense upstream gradient: sampled rows of dW against the oracle, element by element
    if dense_dW_rows:
        H64 = bf16_bits_to_f64(H_bits)
        lse_all, loss_all = orc.dense_forward(H64, W64, labels, IGNORE_INDEX)     # the oracle's own lse of every token
        assert np.abs(lse - lse_all).max() <= TOL_TOKEN and np.abs(loss - loss_all).max() <= TOL_TOKEN
        mean_ref, _ = orc.masked_mean(loss_all, labels, IGNORE_INDEX)
        assert abs(mean_gpu - mean_ref) <= 1e-4 * abs(mean_ref)
        v_idx, never = sampled_vocab_ids(labels, w.V, w.block_v, dense_dW_rows, seed=call)
        dW_ref = orc.rows_dW(v_idx, H64, W64[v_idx], labels, lse_all, dl32, IGNORE_INDEX)
        dW_rows = run.dW[torch.from_numpy(v_idx).cuda()].double().cpu().numpy()
        assert relF(dW_rows, dW_ref) <= TOL_GRAD
        is_never = np.isin(v_idx, never)
        assert is_never.sum() >= dense_dW_rows // 4 and (~is_never).sum() >= dense_dW_rows // 8
        # rows without any one-hot term: the softmax part alone, no rounding of a dominant entry to hide behind
        e_never = relF(dW_rows[is_never], dW_ref[is_never])
        e_targ = relF(dW_rows[~is_never], dW_ref[~is_never])
        print(f"{w.name}: dense-dloss dW rows vs oracle: all {relF(dW_rows, dW_ref):.2e}, "
              f"untargeted {e_never:.2e}, targeted {e_targ:.2e}, rows {len(v_idx)}")
        assert e_never <= TOL_GRAD and e_targ <= TOL_GRAD
        # every single sampled row is right, not only their sum of squares (a row's own norm as the scale)
        row_err = np.linalg.norm(dW_rows - dW_ref, axis=1) / np.maximum(np.linalg.norm(dW_ref, axis=1), 1e-300)
        assert row_err.max() <= 2 * TOL_GRAD, (float(row_err.max()), int(v_idx[row_err.argmax()]))
        del H64
    # ---- sparse upstream gradient: all of dW against the oracle
    dl_sparse = np.zeros(w.T, dtype=np.float32)
    sp = sparse_token_set(w.T, seed=call)
    sp = sp[labels[sp] != IGNORE_INDEX]
    dl_sparse[sp] = (0.5 + np.random.default_rng(call).random(len(sp))).astype(np.float32)
    run.backward(dloss=dl_sparse)
    assert run.bwd_status == 0
    Hs64 = bf16_bits_to_f64(H_bits[sp])
    lse_sp, _, y = orc.rows_forward(Hs64, W64, labels[sp], IGNORE_INDEX)
    G = np.exp(y - lse_sp[:, None])
    del y
    G[np.arange(len(sp)), labels[sp]] -= 1.0
    G *= dl_sparse[sp].astype(np.float64)[:, None]
    dW_ref = G.T @ Hs64                                     # [V, d], exact definition on the sampled tokens
    dW_gpu = run.dW.double().cpu()
    err = float((dW_gpu - torch.from_numpy(dW_ref)).norm() / np.linalg.norm(dW_ref))
    assert err <= TOL_GRAD, err
    never_sp = untargeted_ids(labels[sp], w.V)
    err_never = relF(dW_gpu.numpy()[never_sp], dW_ref[never_sp])
    print(f"{w.name} call {call}: sparse-dloss dW vs oracle: all {err:.2e}, untargeted rows {err_never:.2e}, "
          f"{len(sp)} tokens")
    assert err_never <= TOL_GRAD
    del dW_gpu, dW_ref
    # tokens outside the sample got a zero upstream gradient: their dH rows are exactly zero
    others = np.setdiff1d(np.arange(w.T), sp)[:4096]
    assert not run.dH[torch.from_numpy(others).cuda()].any()
    dH_sp_ref = G @ W64
    dH_sp = run.dH[torch.from_numpy(sp).cuda()].float().cpu().numpy().astype(np.float64)
    assert relF(dH_sp, dH_sp_ref) <= TOL_GRAD
    return run


def test_config3_moe120b_full_size():
    w = WORKLOADS["moe120b"]
    W_bits, W64 = weights("moe120b")
    labels = stream_labels(w)
    check_call(w, 0, W_bits, W64, labels, int((labels != IGNORE_INDEX).sum()), BENCH_T_CHUNK["moe120b"],
               dense_dW_rows=320)


def test_config5_longctx_sampled_calls_and_workspace():
    w = WORKLOADS["longctx"]
    w3 = WORKLOADS["moe120b"]
    T_chunk = BENCH_T_CHUNK["longctx"]
    assert T_chunk == BENCH_T_CHUNK["moe120b"]
    # peak workspace equals config 3's: same (T_chunk, d, block_v); no dependence on V, T or the call count
    assert vp.vp_ce_workspace_bytes(T_chunk, w.d, w.block_v) == vp.vp_ce_workspace_bytes(T_chunk, w3.d, w3.block_v)
    W_bits = make_weights(w)
    W64 = bf16_bits_to_f64(W_bits)
    labels = stream_labels(w)
    assert (labels == IGNORE_INDEX).sum() == 10486
    n_valid_total = int((labels != IGNORE_INDEX).sum())
    Wd = None
    for call in (0, 31, 63):                                 # first, middle, last call of the stream
        run = check_call(w, call, W_bits, W64, labels, n_valid_total, T_chunk, W_dev=Wd, n_sample_tiles=64)
        Wd = run.W
        assert run.ws_bytes == vp.vp_ce_workspace_bytes(T_chunk, w3.d, w3.block_v)


def test_config4_moe667b_full_size():
    w = WORKLOADS["moe667b"]
    W_bits = make_weights(w)
    W64 = bf16_bits_to_f64(W_bits)
    labels = stream_labels(w)
    check_call(w, 0, W_bits, W64, labels, int((labels != IGNORE_INDEX).sum()), BENCH_T_CHUNK["moe667b"],
               n_sample_tiles=128)
