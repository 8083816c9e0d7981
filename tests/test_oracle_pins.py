"""Pins for the float64 oracle: closed forms, invariants, brute force, library special cases.

Each test is chosen so that a plausible mistake in oracle/vpce_oracle.py (a dropped term, a
wrong sign or index, a transposed operand, a wrong rotation) makes it fail.  None of the
expected values comes from the oracle itself or from the CUDA path.
"""
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

from oracle import vpce_oracle as orc
from synth_inputs import (IGNORE_INDEX, WORKLOADS, bf16_bits_to_f64, custom_workload,
                          f32_to_bf16_bits, make_batch, stream_labels, zipf_cdf)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_problem(T=24, d=16, V=50, seed=0, ignore_frac=0.25, w_std=0.5):
    w = custom_workload("small", T=T, d=d, V=V, block_v=16, T_chunk=8, w_std=w_std,
                        labels="uniform", ignore_frac=ignore_frac, seed=seed)
    b = make_batch(w)
    return bf16_bits_to_f64(b.H_bits), bf16_bits_to_f64(b.W_bits), b.labels


# ------------------------------------------------------------------ closed forms (P1, P2, P7)
def test_zero_weight_gives_log_V_and_closed_form_dW():
    H, W, lab = small_problem()
    W0 = np.zeros_like(W)
    V = W.shape[0]
    lse, loss = orc.dense_forward(H, W0, lab, IGNORE_INDEX)
    valid = lab != IGNORE_INDEX
    assert np.all(lse == math.log(V))
    assert np.all(loss[valid] == math.log(V)) and np.all(loss[~valid] == 0.0)
    dl = orc.default_dloss(lab, IGNORE_INDEX)
    dH, dW = orc.dense_backward(H, W0, lab, None, IGNORE_INDEX)
    assert np.all(dH == 0.0)
    expect = np.tile((dl[:, None] * H).sum(0) / V, (V, 1))
    for n in np.nonzero(valid)[0]:
        expect[lab[n]] -= dl[n] * H[n]
    np.testing.assert_allclose(dW, expect, rtol=0, atol=1e-13)


def test_zero_hidden_gives_closed_form_dH():
    H, W, lab = small_problem(seed=3)
    H0 = np.zeros_like(H)
    V = W.shape[0]
    lse, loss = orc.dense_forward(H0, W, lab, IGNORE_INDEX)
    assert np.all(lse == math.log(V))
    dl = orc.default_dloss(lab, IGNORE_INDEX)
    dH, dW = orc.dense_backward(H0, W, lab, None, IGNORE_INDEX)
    assert np.all(dW == 0.0)
    expect = np.zeros_like(H)
    for n in range(H.shape[0]):
        if lab[n] != IGNORE_INDEX:
            expect[n] = dl[n] * (W.mean(0) - W[lab[n]])
    np.testing.assert_allclose(dH, expect, rtol=0, atol=1e-13)


def test_V1_and_V2_textbook_cases():
    rng = np.random.default_rng(0)
    H = rng.standard_normal((5, 4))
    W1 = rng.standard_normal((1, 4))
    lab = np.zeros(5, dtype=np.int32)
    lse, loss = orc.dense_forward(H, W1, lab)
    np.testing.assert_allclose(loss, 0.0, atol=1e-13)
    dH, dW = orc.dense_backward(H, W1, lab)
    np.testing.assert_allclose(dH, 0.0, atol=1e-13)
    np.testing.assert_allclose(dW, 0.0, atol=1e-13)
    W2 = rng.standard_normal((2, 4))
    lab2 = np.array([0, 1, 1, 0, 1], dtype=np.int32)
    _, loss2 = orc.dense_forward(H, W2, lab2)
    y = H @ W2.T
    gap = y[np.arange(5), lab2] - y[np.arange(5), 1 - lab2]
    np.testing.assert_allclose(loss2, np.log1p(np.exp(-gap)), rtol=1e-12)


# ------------------------------------------------------------------ invariants (P3, P8, P10)
def test_residual_rows_sum_to_zero():
    H, W, lab = small_problem(seed=5)
    dH, dW = orc.dense_backward(H, W, lab)
    # sum_v G[n, v] = 0 for every token, hence the column sums of dW vanish ...
    np.testing.assert_allclose(dW.sum(0), 0.0, atol=1e-12)
    # ... and dH[n] = dloss_n (sum_v p_v W_v - W_t)
    dl = orc.default_dloss(lab, IGNORE_INDEX)
    p = scipy.special.softmax(H @ W.T, axis=1)
    for n in range(H.shape[0]):
        e = np.zeros(W.shape[1]) if lab[n] == IGNORE_INDEX else dl[n] * (p[n] @ W - W[lab[n]])
        np.testing.assert_allclose(dH[n], e, atol=1e-12)


def test_logit_shift_invariance_and_large_logits():
    H, W, lab = small_problem(seed=7, w_std=1.0)
    w0 = np.random.default_rng(1).standard_normal(W.shape[1]) * 300.0
    lse, loss = orc.dense_forward(H, W, lab)
    lse_s, loss_s = orc.dense_forward(H, W + w0, lab)
    np.testing.assert_allclose(lse_s - lse, H @ w0, rtol=1e-10, atol=1e-8)
    np.testing.assert_allclose(loss_s, loss, atol=1e-8)
    assert np.isfinite(lse_s).all() and np.abs(H @ w0).max() > 1e3
    dH, dW = orc.dense_backward(H, W, lab)
    dH_s, dW_s = orc.dense_backward(H, W + w0, lab)
    np.testing.assert_allclose(dH_s, dH, atol=1e-9)
    np.testing.assert_allclose(dW_s, dW, atol=1e-9)


def test_ignored_tokens_touch_only_their_own_lse():
    H, W, lab = small_problem(seed=9)
    ign = lab == IGNORE_INDEX
    assert ign.any() and (~ign).any()
    H2 = H.copy()
    H2[ign] = np.random.default_rng(2).standard_normal((ign.sum(), H.shape[1]))
    a = orc.forward_backward(H, W, lab)
    b = orc.forward_backward(H2, W, lab)
    assert np.array_equal(a["loss"], b["loss"]) and a["mean"] == b["mean"]
    assert np.array_equal(a["lse"][~ign], b["lse"][~ign])
    assert not np.array_equal(a["lse"][ign], b["lse"][ign])
    assert np.array_equal(a["dW"], b["dW"]) and np.array_equal(a["dH"], b["dH"])
    assert np.all(a["dH"][ign] == 0.0)


def test_all_ignored_gives_zero_mean_and_gradients():
    H, W, lab = small_problem(seed=11)
    lab = np.full_like(lab, IGNORE_INDEX)
    r = orc.forward_backward(H, W, lab)
    assert r["mean"] == 0.0 and r["n_valid"] == 0
    assert not r["dH"].any() and not r["dW"].any() and not r["loss"].any()
    assert np.isfinite(r["lse"]).all()


def test_out_of_range_label_raises():
    H, W, lab = small_problem(seed=12)
    lab = lab.copy()
    lab[0] = W.shape[0]
    with pytest.raises(ValueError):
        orc.dense_forward(H, W, lab)
    lab[0] = -1
    with pytest.raises(ValueError):
        orc.dense_backward(H, W, lab)


# ------------------------------------------------------------------ brute force (P5, naive loops)
def test_naive_python_loops_match_dense():
    H, W, lab = small_problem(T=6, d=5, V=11, seed=13)
    lse, loss = orc.dense_forward(H, W, lab)
    dH, dW = orc.dense_backward(H, W, lab)
    nl, nloss, ndH, ndW = orc.naive_forward_backward(H.tolist(), W.tolist(), lab.tolist())
    np.testing.assert_allclose(lse, nl, rtol=1e-12)
    np.testing.assert_allclose(loss, nloss, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dH, ndH, atol=1e-13)
    np.testing.assert_allclose(dW, ndW, atol=1e-13)


@pytest.mark.parametrize("explicit_dloss", [False, True])
def test_central_finite_differences(explicit_dloss):
    rng = np.random.default_rng(17)
    T, d, V = 4, 3, 7
    H = rng.standard_normal((T, d))
    W = rng.standard_normal((V, d))
    lab = np.array([2, IGNORE_INDEX, 6, 0], dtype=np.int32)
    dl = rng.random(T) if explicit_dloss else None

    def objective(Hx, Wx):
        # written from the definition with scipy's logsumexp, not with the oracle
        y = Hx @ Wx.T
        per = np.array([0.0 if t == IGNORE_INDEX else scipy.special.logsumexp(y[n]) - y[n, t]
                        for n, t in enumerate(lab)])
        if dl is None:
            return per.sum() / (lab != IGNORE_INDEX).sum()
        return float((dl * per).sum())

    dH, dW = orc.dense_backward(H, W, lab, dl)
    eps = 1e-6
    for (n, k) in [(0, 0), (1, 1), (2, 2), (3, 1)]:
        Hp, Hm = H.copy(), H.copy()
        Hp[n, k] += eps
        Hm[n, k] -= eps
        fd = (objective(Hp, W) - objective(Hm, W)) / (2 * eps)
        assert abs(fd - dH[n, k]) < 1e-8
    for v in range(V):
        for k in range(d):
            Wp, Wm = W.copy(), W.copy()
            Wp[v, k] += eps
            Wm[v, k] -= eps
            fd = (objective(H, Wp) - objective(H, Wm)) / (2 * eps)
            assert abs(fd - dW[v, k]) < 1e-8


# ------------------------------------------------------------------ library special case (P6)
def test_matches_torch_cross_entropy_and_autograd():
    H, W, lab = small_problem(T=40, d=24, V=97, seed=19)
    Ht = torch.tensor(H, dtype=torch.float64, requires_grad=True)
    Wt = torch.tensor(W, dtype=torch.float64, requires_grad=True)
    logits = Ht @ Wt.T
    per = torch.nn.functional.cross_entropy(logits, torch.tensor(lab, dtype=torch.long),
                                            ignore_index=IGNORE_INDEX, reduction="none")
    mean = torch.nn.functional.cross_entropy(logits, torch.tensor(lab, dtype=torch.long),
                                             ignore_index=IGNORE_INDEX, reduction="mean")
    mean.backward()
    r = orc.forward_backward(H, W, lab)
    np.testing.assert_allclose(r["loss"], per.detach().numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(r["lse"], torch.logsumexp(logits, 1).detach().numpy(), rtol=1e-12)
    assert abs(r["mean"] - mean.item()) < 1e-12
    np.testing.assert_allclose(r["dH"], Ht.grad.numpy(), atol=1e-13)
    np.testing.assert_allclose(r["dW"], Wt.grad.numpy(), atol=1e-13)


# ------------------------------------------------------------------ Algorithm 3 (P4, rotation, ownership)
def test_rotation_order_matches_formula_fixture():
    with open(os.path.join(GOLDEN, "rotation_order.txt")) as f:
        rows = [ln for ln in f if ln.strip() and not ln.startswith("#")]
    assert rows
    for ln in rows:
        left, right = ln.split(":")
        P, r = (int(x) for x in left.split())
        assert list(orc.shard_order(r, P)) == [int(x) for x in right.split()]


@pytest.mark.parametrize("block_v,T_chunk,base", [(16, 8, 0), (7, 5, 3), (50, 24, 1), (64, 100, 9),
                                                  (1, 24, 0), (13, 1, 2)])
def test_blocked_fold_equals_dense(block_v, T_chunk, base):
    H, W, lab = small_problem(seed=23)
    lse, loss = orc.dense_forward(H, W, lab)
    for direction in (-1, +1):
        for off in (0, 2):
            l2, s2, gathers = orc.ring_fold_forward(H, W, lab, block_v, T_chunk, base, IGNORE_INDEX,
                                                    direction, off)
            np.testing.assert_allclose(l2, lse, rtol=1e-12)
            np.testing.assert_allclose(s2, loss, rtol=1e-12, atol=1e-13)
            # exclusive target-column ownership: exactly one meeting supplies y_t
            assert np.array_equal(gathers, (lab != IGNORE_INDEX).astype(np.int64))


def test_fold_single_step_by_hand():
    # one token, strip [1, 3], state (m=2, z=0.5): m' = 3, z' = e^{-1} 0.5 + e^{-2} + 1
    S = (np.array([2.0]), np.array([0.5]), np.array([0.0]))
    (m, z, y), own = orc.fold(S, np.array([[1.0, 3.0]]), np.array([11]), 10, 12)
    assert m[0] == 3.0
    assert abs(z[0] - (math.exp(-1) * 0.5 + math.exp(-2) + 1.0)) < 1e-15
    assert y[0] == 3.0 and own[0]
    # from the initial state (-inf, 0, 0) no NaN appears
    S0 = (np.array([-np.inf]), np.array([0.0]), np.array([0.0]))
    (m, z, y), own = orc.fold(S0, np.array([[1.0, 3.0]]), np.array([5]), 10, 12)
    assert m[0] == 3.0 and abs(z[0] - (1 + math.exp(-2))) < 1e-15 and y[0] == 0.0 and not own[0]


@pytest.mark.parametrize("block_v,T_chunk,base", [(16, 8, 0), (7, 5, 3), (64, 100, 2)])
def test_ring_backward_equals_dense(block_v, T_chunk, base):
    H, W, lab = small_problem(seed=29)
    dl = np.random.default_rng(3).random(H.shape[0])
    lse, _ = orc.dense_forward(H, W, lab)
    for dloss in (None, dl):
        dH, dW = orc.dense_backward(H, W, lab, dloss)
        rH, rW = orc.ring_backward(H, W, lab, lse, block_v, T_chunk, base, dloss)
        np.testing.assert_allclose(rH, dH, atol=1e-12)
        np.testing.assert_allclose(rW, dW, atol=1e-12)


# ------------------------------------------------------------------ sampled-output helpers
def test_sampled_rows_equal_dense():
    H, W, lab = small_problem(T=30, d=12, V=70, seed=31)
    dl = np.random.default_rng(4).random(H.shape[0])
    lse, loss = orc.dense_forward(H, W, lab)
    dH, dW = orc.dense_backward(H, W, lab, dl)
    rows = np.array([0, 7, 13, 29])
    l, s, _ = orc.rows_forward(H[rows], W, lab[rows], v_slab=16)
    np.testing.assert_allclose(l, lse[rows], rtol=1e-12)
    np.testing.assert_allclose(s, loss[rows], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(orc.rows_dH(H[rows], W, lab[rows], dl[rows], v_slab=16), dH[rows], atol=1e-12)
    vs = np.array([0, 3, int(lab[lab != IGNORE_INDEX][0]), 69])
    np.testing.assert_allclose(orc.rows_dW(vs, H, W[vs], lab, lse, dl), dW[vs], atol=1e-12)


# ------------------------------------------------------------------ statistics + paper arithmetic (P9, P11)
def test_expected_loss_of_gaussian_inputs():
    # For y ~ N(0, s^2) i.i.d. over a large vocabulary, E[loss] ~ ln V + s^2 / 2 with s^2 = d Var(W).
    w = WORKLOADS["tiny"]
    b = make_batch(w)
    H, W = bf16_bits_to_f64(b.H_bits), bf16_bits_to_f64(b.W_bits)
    _, loss = orc.dense_forward(H, W, b.labels)
    s2 = w.d * w.w_std ** 2
    assert abs(loss.mean() - (math.log(w.V) + s2 / 2)) < 0.15


def test_paper_memory_table_arithmetic():
    vals = {}
    with open(os.path.join(GOLDEN, "ringdtp_memory_table.txt")) as f:
        for ln in f:
            if ln.strip() and not ln.startswith("#"):
                k, v = ln.split()
                vals[k] = float(v)
    N, Hd, V, b = int(vals["N"]), int(vals["H"]), int(vals["V"]), int(vals["bytes_per_value"])
    gib = 2.0 ** 30
    assert abs(Hd * V * b / gib - vals["projection_weight_standard"]) < 5e-5
    assert abs(Hd * V * b / 4 / gib - vals["projection_weight_P4"]) < 1e-4
    assert abs(Hd * V * b / 8 / gib - vals["projection_weight_P8"]) < 1e-4
    # a dense forward+backward holds three N x V arrays: logits, log-softmax, logit gradient
    assert abs(3 * N * V * b / gib - vals["increment_over_resident_standard"]) < 2e-4
    w = custom_workload("paper", T=N, d=Hd, V=V, block_v=V // 8, T_chunk=N)
    assert w.logits_bytes_fp32 == N * V * 4


# ------------------------------------------------------------------ input generator (host logic)
def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -2.5, 0.0, 3.14159], dtype=np.float32)
    bits = f32_to_bf16_bits(x)
    ref = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    big = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    assert np.array_equal(f32_to_bf16_bits(big),
                          torch.tensor(big).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


def test_workload_recipe_counts_and_determinism():
    expect_ignored = {"tiny": 0, "mid": 410, "moe120b": 819, "moe667b": 1311, "longctx": 10486}
    for name, w in WORKLOADS.items():
        assert w.n_ignored == expect_ignored[name]
    w = WORKLOADS["mid"]
    lab = stream_labels(w)
    assert (lab == IGNORE_INDEX).sum() == 410
    assert lab[lab != IGNORE_INDEX].min() >= 0 and lab.max() < w.V
    assert np.array_equal(lab, stream_labels(w))
    cdf = zipf_cdf(w.V, 1.1)
    assert abs(cdf[0] - 0.142) < 2e-3 and abs(cdf[8191] - 0.925) < 2e-3
    # empirical mass of id 0 close to the law's
    assert abs((lab == 0).mean() / 0.9 - cdf[0]) < 0.02
    assert WORKLOADS["moe120b"].P == 25 and WORKLOADS["moe667b"].P == 16
    assert WORKLOADS["longctx"].T_stream == 1048576
    t = make_batch(WORKLOADS["tiny"])
    t2 = make_batch(WORKLOADS["tiny"])
    assert t.checksums() == t2.checksums()
    Hf = bf16_bits_to_f64(t.H_bits)
    assert abs(Hf.std() - 1.0) < 0.02 and abs(bf16_bits_to_f64(t.W_bits).std() - 1 / 16) < 0.002
