"""The torch.autograd front end against plain PyTorch float32 cross-entropy of the same operation and
against the float64 oracle."""
import numpy as np
import pytest
import torch

import paper_2609_14306_b200 as vp
from oracle import vpce_oracle as orc
from synth_inputs import IGNORE_INDEX, bf16_bits_to_f64, custom_workload, make_batch
from vpce_testlib import TOL_GRAD, TOL_TOKEN, relF, to_dev_bf16

pytestmark = pytest.mark.gpu


def test_autograd_mean_loss_matches_pytorch_and_oracle():
    w = custom_workload("ag", T=640, d=256, V=5000, block_v=1024, T_chunk=256, w_std=0.0625,
                        labels="zipf", ignore_frac=0.1, seed=51)
    b = make_batch(w)
    H = to_dev_bf16(b.H_bits).requires_grad_(True)
    W = to_dev_bf16(b.W_bits).requires_grad_(True)
    lab = torch.from_numpy(b.labels).cuda()
    loss = vp.vocab_proj_cross_entropy_mean(H, W, lab, block_v=w.block_v, T_chunk=w.T_chunk)
    loss.backward()
    # plain PyTorch fp32 reference of the same op on the same bf16 values
    Hr = H.detach().float().requires_grad_(True)
    Wr = W.detach().float().requires_grad_(True)
    ref = torch.nn.functional.cross_entropy(Hr @ Wr.T, lab.long(), ignore_index=IGNORE_INDEX)
    ref.backward()
    assert abs(loss.item() - ref.item()) <= 1e-4 * abs(ref.item())
    assert relF(H.grad.float().cpu().numpy(), Hr.grad.cpu().numpy().astype(np.float64)) <= TOL_GRAD
    assert relF(W.grad.float().cpu().numpy(), Wr.grad.cpu().numpy().astype(np.float64)) <= TOL_GRAD
    o = orc.forward_backward(bf16_bits_to_f64(b.H_bits), bf16_bits_to_f64(b.W_bits), b.labels)
    assert abs(loss.item() - o["mean"]) <= 1e-4 * abs(o["mean"])
    assert relF(H.grad.float().cpu().numpy(), o["dH"]) <= TOL_GRAD


def test_autograd_per_token_loss_with_fp32_accumulation_buffer():
    w = custom_workload("ag2", T=384, d=128, V=2000, block_v=512, T_chunk=128, w_std=0.09,
                        labels="uniform", ignore_frac=0.05, seed=52)
    b = make_batch(w)
    H = to_dev_bf16(b.H_bits).requires_grad_(True)
    W = to_dev_bf16(b.W_bits).requires_grad_(True)
    lab = torch.from_numpy(b.labels).cuda()
    dl = np.random.default_rng(0).random(w.T).astype(np.float32)
    main_grad = torch.zeros(w.V, w.d, dtype=torch.float32, device="cuda")
    per_tok = vp.vocab_proj_cross_entropy(H, W, lab, block_v=w.block_v, T_chunk=w.T_chunk, dW_accum=main_grad)
    (per_tok * torch.from_numpy(dl).cuda()).sum().backward()
    o = orc.forward_backward(bf16_bits_to_f64(b.H_bits), bf16_bits_to_f64(b.W_bits), b.labels, dl.astype(np.float64))
    assert np.abs(per_tok.detach().cpu().numpy() - o["loss"]).max() <= TOL_TOKEN
    assert W.grad is None                                     # the weight gradient went to the fp32 buffer
    assert relF(main_grad.cpu().numpy(), o["dW"]) <= TOL_GRAD
    assert relF(H.grad.float().cpu().numpy(), o["dH"]) <= TOL_GRAD


def test_autograd_second_backward_and_frozen_weight():
    w = custom_workload("ag3", T=256, d=128, V=1500, block_v=512, T_chunk=128, w_std=0.09,
                        labels="uniform", ignore_frac=0.05, seed=53)
    b = make_batch(w)
    o = orc.forward_backward(bf16_bits_to_f64(b.H_bits), bf16_bits_to_f64(b.W_bits), b.labels)
    lab = torch.from_numpy(b.labels).cuda()
    # a graph that is walked twice (retain_graph): the second backward allocates its own workspace
    H = to_dev_bf16(b.H_bits).requires_grad_(True)
    W = to_dev_bf16(b.W_bits).requires_grad_(True)
    loss = vp.vocab_proj_cross_entropy_mean(H, W, lab, block_v=w.block_v, T_chunk=w.T_chunk)
    loss.backward(retain_graph=True)
    g1 = H.grad.clone()
    H.grad = None
    loss.backward()
    assert torch.equal(g1.view(torch.int16), H.grad.view(torch.int16))
    assert relF(H.grad.float().cpu().numpy(), o["dH"]) <= TOL_GRAD
    # a frozen projection weight: only the input gradient is computed (the weight-gradient GEMM is skipped)
    H2 = to_dev_bf16(b.H_bits).requires_grad_(True)
    W2 = to_dev_bf16(b.W_bits)
    n0 = vp.vp_ce_launch_count()
    vp.vocab_proj_cross_entropy_mean(H2, W2, lab, block_v=w.block_v, T_chunk=w.T_chunk).backward()
    launches_frozen = vp.vp_ce_launch_count() - n0
    assert relF(H2.grad.float().cpu().numpy(), o["dH"]) <= TOL_GRAD
    # and the other way round: only the weight gradient
    H3 = to_dev_bf16(b.H_bits)
    W3 = to_dev_bf16(b.W_bits).requires_grad_(True)
    n0 = vp.vp_ce_launch_count()
    vp.vocab_proj_cross_entropy_mean(H3, W3, lab, block_v=w.block_v, T_chunk=w.T_chunk).backward()
    launches_weight_only = vp.vp_ce_launch_count() - n0
    assert relF(W3.grad.float().cpu().numpy(), o["dW"]) <= TOL_GRAD
    chunks = w.T // w.T_chunk
    meetings = chunks * w.P
    n0 = vp.vp_ce_launch_count()
    vp.vocab_proj_cross_entropy_mean(H, W, lab, block_v=w.block_v, T_chunk=w.T_chunk).backward()
    both = vp.vp_ce_launch_count() - n0
    # without dW: no weight-gradient GEMM per (chunk, shard) and no one-hot scatter (two launches) per chunk
    assert both == launches_frozen + meetings + 2 * chunks
    # without dH: no input-gradient GEMM per (chunk, shard) and no finishing pass over the accumulator per chunk
    assert both == launches_weight_only + meetings + chunks


def test_autograd_empty_batch():
    d, V = 64, 512
    H = torch.empty(0, d, dtype=torch.bfloat16, device="cuda", requires_grad=True)
    W = (torch.randn(V, d, device="cuda") * 0.1).to(torch.bfloat16).requires_grad_(True)
    lab = torch.empty(0, dtype=torch.int64, device="cuda")
    loss = vp.vocab_proj_cross_entropy_mean(H, W, lab, block_v=256)
    assert float(loss.detach()) == 0.0                         # no valid token: mean 0 (the documented rule)
    loss.backward()
    assert H.grad.shape == (0, d)
    assert W.grad is not None and not W.grad.any()             # an empty batch contributes nothing
