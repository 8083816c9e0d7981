"""GPU parity of the FP32-input (TF32 tensor core) entry points against the float64 oracle on the same
float32 inputs.  As on the bf16 path the inputs are rounded to what the tensor core multiplies exactly
(TF32-representable float32), so the acceptance tolerances test the kernel's arithmetic; one more test
feeds unrounded float32 and bounds the cost of the TF32 input precision itself."""
import numpy as np
import pytest
import torch

import paper_2609_14306_b200 as vp
from oracle import vpce_oracle as orc
from synth_inputs import (IGNORE_INDEX, PROFILE_WORKLOADS, custom_workload, make_hidden_f32, make_weights_f32,
                          stream_labels)
from vpce_testlib import TOL_GRAD, TOL_TOKEN, relF

pytestmark = pytest.mark.gpu


def run_f32(w, base=0, dloss=None, tf32_inputs=True, tol_token=TOL_TOKEN):
    H = make_hidden_f32(w, tf32=tf32_inputs)
    W = make_weights_f32(w, tf32=tf32_inputs)
    lab = stream_labels(w)[:w.T]
    Hd, Wd = torch.from_numpy(H).cuda(), torch.from_numpy(W).cuda()
    ld = torch.from_numpy(lab).cuda()
    nbytes = vp.vp_ce_workspace_bytes_f32(w.T_chunk, w.d, w.block_v)
    assert nbytes > 0
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    loss = torch.full((w.T,), float("nan"), device="cuda")
    lse = torch.full((w.T,), float("nan"), device="cuda")
    dH = torch.full((w.T, w.d), float("nan"), device="cuda")
    dW = torch.full((w.V, w.d), float("nan"), device="cuda")
    vp.vp_ce_forward_f32(Hd, Wd, ld, w.block_v, IGNORE_INDEX, loss, lse, w.T_chunk, base, ws)
    dl = None if dloss is None else torch.from_numpy(dloss).cuda()
    vp.vp_ce_backward_f32(Hd, Wd, ld, lse, dl, dH, dW, w.block_v, IGNORE_INDEX, w.T_chunk, base, False, ws)
    torch.cuda.synchronize()
    assert vp.vp_ce_device_status(ws) == 0
    ref = orc.forward_backward(H.astype(np.float64), W.astype(np.float64), lab,
                               None if dloss is None else dloss.astype(np.float64), IGNORE_INDEX)
    e = {"lse": float(np.abs(lse.cpu().numpy() - ref["lse"]).max()),
         "loss": float(np.abs(loss.cpu().numpy() - ref["loss"]).max()),
         "dH": relF(dH.cpu().numpy(), ref["dH"]), "dW": relF(dW.cpu().numpy(), ref["dW"])}
    print(w.name, e)
    assert e["lse"] <= tol_token and e["loss"] <= tol_token and e["dH"] <= TOL_GRAD and e["dW"] <= TOL_GRAD, e
    return e


@pytest.mark.parametrize("T,d,V,block_v,T_chunk", [
    (512, 256, 2048, 512, 256),
    (300, 96, 1000, 512, 128),      # ragged tokens, ragged last shard, d = 3 k-blocks of 32
    (128, 32, 300, 256, 128),       # one 128-row tile (the pair's second CTA is all padding), one k-block
    (384, 2880, 1536, 512, 384),    # the 120B hidden width: 11 full output tiles + a narrow one
])
def test_f32_shapes(T, d, V, block_v, T_chunk):
    w = custom_workload(f"f32_{T}x{d}x{V}", T=T, d=d, V=V, block_v=block_v, T_chunk=T_chunk,
                        w_std=1.0 / np.sqrt(d), labels="zipf", ignore_frac=0.06, seed=T + d)
    run_f32(w, base=2)


def test_f32_unrounded_inputs_cost_of_tf32():
    # plain float32 inputs: the tensor core drops 13 mantissa bits of every input, ~2^-11 per product;
    # with unit-variance logits that is ~1e-3 on a logit, so the per-token budget here is 1e-2
    w = custom_workload("f32_raw", T=512, d=256, V=2048, block_v=512, T_chunk=256, w_std=1.0 / 16,
                        labels="zipf", ignore_frac=0.06, seed=99)
    e = run_f32(w, tf32_inputs=False, tol_token=1e-2)
    assert e["lse"] > 1e-5                                  # the inputs really were not TF32-representable


def test_tf32_rounding_helper():
    from synth_inputs import f32_round_to_tf32
    x = np.array([1.0, 1.0 + 2 ** -11, 1.0 + 2 ** -10, 1.0 + 3 * 2 ** -11, -3.14159, 0.0], dtype=np.float32)
    r = f32_round_to_tf32(x)
    assert (r.view(np.uint32) & 0x1FFF == 0).all()
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == np.float32(1.0 + 2 ** -10) and r[3] == np.float32(1.0 + 2 ** -9)
    assert np.abs(r - x).max() <= 2 ** -10


def test_f32_rejects_unsupported_width():
    assert vp.vp_ce_workspace_bytes_f32(128, 40, 256) == 0      # d % 32
    assert vp.vp_ce_workspace_bytes_f32(128, 64, 256) > 0


def test_paper_shape_full_size_sampled():
    """The shape of the paper's isolated benchmark (App. C / Table 2: N = 16384, H = 7168, V = 200000, P = 8) with
    FP32 inputs, in the launch configuration the benchmark times (block_v = 25088, one chunk).  Sampled as in the
    bf16 full-size tests: lse / loss / dH rows of one token per 128-token tile; with an upstream gradient that is
    non-zero on a sparse token set (one token per 64-token k-block plus one whole tile) ALL of dW and those tokens'
    dH rows; the column sums of dW under the dense mean gradient."""
    w = PROFILE_WORKLOADS["papershape"]
    H = make_hidden_f32(w)
    W = make_weights_f32(w)
    lab = stream_labels(w)[:w.T]
    assert H.shape == (16384, 7168) and W.shape == (200000, 7168) and -(-w.V // w.block_v) == 8

    def W64(v0, v1):
        return W[v0:v1].astype(np.float64)
    W_slabs = (W64, w.V)                                     # the oracle's row helpers accept a slab getter

    Hd, Wd, ld = torch.from_numpy(H).cuda(), torch.from_numpy(W).cuda(), torch.from_numpy(lab).cuda()
    ws = torch.empty(vp.vp_ce_workspace_bytes_f32(w.T_chunk, w.d, w.block_v), dtype=torch.uint8, device="cuda")
    loss = torch.full((w.T,), float("nan"), device="cuda")
    lse = torch.full((w.T,), float("nan"), device="cuda")
    dH = torch.full((w.T, w.d), float("nan"), device="cuda")
    dW = torch.full((w.V, w.d), float("nan"), device="cuda")
    vp.vp_ce_forward_f32(Hd, Wd, ld, w.block_v, IGNORE_INDEX, loss, lse, w.T_chunk, 0, ws)
    vp.vp_ce_backward_f32(Hd, Wd, ld, lse, None, dH, dW, w.block_v, IGNORE_INDEX, w.T_chunk, 0, False, ws)
    torch.cuda.synchronize()
    assert vp.vp_ce_device_status(ws) == 0
    # ---- dense mean gradient: sampled tokens
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([np.arange(w.T // 128) * 128 + rng.integers(0, 128, size=w.T // 128), [0, w.T - 1]]))
    Hr = H[rows].astype(np.float64)
    lse_ref, loss_ref, _ = orc.rows_forward(Hr, W_slabs, lab[rows], IGNORE_INDEX)
    lse_h, loss_h = lse.cpu().numpy().astype(np.float64), loss.cpu().numpy().astype(np.float64)
    assert np.isfinite(lse_h).all() and np.isfinite(loss_h).all()
    assert np.abs(lse_h[rows] - lse_ref).max() <= TOL_TOKEN and np.abs(loss_h[rows] - loss_ref).max() <= TOL_TOKEN
    n_valid = int((lab != IGNORE_INDEX).sum())
    dl = np.full(len(rows), np.float64(np.float32(1.0 / n_valid)))
    dH_ref = orc.rows_dH(Hr, W_slabs, lab[rows], dl, IGNORE_INDEX)
    ridx = torch.from_numpy(rows).cuda()
    assert relF(dH[ridx].cpu().numpy().astype(np.float64), dH_ref) <= TOL_GRAD
    colsum = dW.double().sum(0)
    assert float(colsum.norm() / dW.double().norm()) < 5e-4
    del colsum
    # ---- sparse upstream gradient: every element of dW
    sp = np.unique(np.concatenate([np.arange(w.T // 64) * 64 + rng.integers(0, 64, size=w.T // 64),
                                   np.arange(37 * 128, 38 * 128), [0, w.T - 1]]))
    dls = np.zeros(w.T, dtype=np.float32)
    dls[sp] = (0.5 + rng.random(len(sp))).astype(np.float32)
    vp.vp_ce_backward_f32(Hd, Wd, ld, lse, torch.from_numpy(dls).cuda(), dH, dW, w.block_v, IGNORE_INDEX, w.T_chunk,
                          0, False, ws)
    torch.cuda.synchronize()
    assert vp.vp_ce_device_status(ws) == 0
    Hs = H[sp].astype(np.float64)
    lse_sp, _, y = orc.rows_forward(Hs, W_slabs, lab[sp], IGNORE_INDEX)
    G = np.exp(y - lse_sp[:, None])
    del y
    G[np.arange(len(sp)), lab[sp]] -= 1.0
    G *= dls[sp].astype(np.float64)[:, None]
    num = den = 0.0
    dH_sp_ref = np.zeros((len(sp), w.d))
    for v0 in range(0, w.V, 20000):                          # slab by slab: the full float64 dW never exists on the host
        v1 = min(w.V, v0 + 20000)
        ref = G[:, v0:v1].T @ Hs
        got = dW[v0:v1].cpu().numpy().astype(np.float64)
        num += float(((got - ref) ** 2).sum())
        den += float((ref ** 2).sum())
        dH_sp_ref += G[:, v0:v1] @ W64(v0, v1)
    err = (num / den) ** 0.5
    print(f"papershape tf32: sparse-dloss dW vs oracle {err:.2e} over {len(sp)} tokens")
    assert err <= TOL_GRAD
    assert relF(dH[torch.from_numpy(sp).cuda()].cpu().numpy().astype(np.float64), dH_sp_ref) <= TOL_GRAD
    others = np.setdiff1d(np.arange(w.T), sp)[:4096]
    assert not dH[torch.from_numpy(others).cuda()].any()
