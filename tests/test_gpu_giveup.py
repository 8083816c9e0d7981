"""The give-up path of the kernels' bounded waits, exercised without any invalid access.

Every wait inside the GEMM kernels has a time limit.  The library's test hook makes ONE copy of one launch
"get lost" on the host's request (the producer simply does not issue it), so a "full" barrier never completes:
the MMA issuer's wait runs out, the CTA (or CTA pair) stops taking work, waits for what it has in flight, frees
its tensor memory and returns, and the status word reports VPCE_DEV_WAIT_EXPIRED.  The tests check that the call
returns promptly, that the status bit is set, and that the very next call on the same workspace is correct."""
import time

import numpy as np
import pytest
import torch

import paper_2609_14306_b200 as vp
from oracle import vpce_oracle as orc
from synth_inputs import IGNORE_INDEX, bf16_bits_to_f64, custom_workload, make_batch
from vpce_testlib import TOL_GRAD, TOL_TOKEN, DeviceRun, relF, to_dev_bf16

pytestmark = pytest.mark.gpu

WAIT_EXPIRED = 2
LIMIT_NS = 2_000_000          # 2 ms for these tests; the default is 2 s


def _problem(pair):
    # pair kernels need at least two 128-row tiles per launch; a single tile selects the one-CTA kernel
    T, T_chunk = (512, 256) if pair else (128, 128)
    w = custom_workload("giveup", T=T, d=256, V=1024, block_v=512, T_chunk=T_chunk, w_std=0.0625,
                        labels="zipf", ignore_frac=0.05, seed=61)
    b = make_batch(w)
    ref = orc.forward_backward(bf16_bits_to_f64(b.H_bits), bf16_bits_to_f64(b.W_bits), b.labels)
    return w, b, ref


@pytest.mark.parametrize("kind,pair,ranks", [
    (0, True, 1),     # forward strip, CTA pair, the leader's copy is lost
    (0, True, 2),     # ... the second CTA's copy is lost (the leader's barrier gets half its bytes)
    (1, True, 3),     # backward strip, both CTAs
    (2, True, 2),     # input-gradient GEMM
    (3, True, 1),     # weight-gradient GEMM
    (0, False, 1),    # one-CTA kernels
    (1, False, 1),
    (2, False, 1),
])
def test_lost_copy_expires_the_waits_and_the_next_call_is_clean(kind, pair, ranks):
    w, b, ref = _problem(pair)
    run = DeviceRun(b.H_bits, b.W_bits, b.labels, w.block_v, w.T_chunk, chunk_index_base=1)
    prev = vp.vp_ce_set_wait_limit_ns(LIMIT_NS)
    try:
        assert prev == 2_000_000_000
        if kind == 0:
            vp.vp_ce_debug_drop_copy(kind, 1, ranks)
            t0 = time.perf_counter()
            run.forward()
            dt = time.perf_counter() - t0
            status = run.fwd_status
        else:
            run.forward()
            assert run.fwd_status == 0
            vp.vp_ce_debug_drop_copy(kind, 1, ranks)
            t0 = time.perf_counter()
            run.backward()
            dt = time.perf_counter() - t0
            status = run.bwd_status
    finally:
        vp.vp_ce_debug_drop_copy(-1)
        vp.vp_ce_set_wait_limit_ns(prev)
    assert status & WAIT_EXPIRED, status
    assert dt < 1.0, dt                       # a few wait limits, not the 2 s default and not a hang
    # the context is intact and the same workspace serves a normal call right away
    run.forward().backward()
    assert run.fwd_status == 0 and run.bwd_status == 0
    assert np.abs(run.np_lse() - ref["lse"]).max() <= TOL_TOKEN
    assert np.abs(run.np_loss() - ref["loss"]).max() <= TOL_TOKEN
    assert relF(run.np_dH(), ref["dH"]) <= TOL_GRAD and relF(run.np_dW(), ref["dW"]) <= TOL_GRAD


def test_lost_copy_in_the_static_scratch_forward_reports_through_its_status_output():
    w, b, ref = _problem(pair=False)
    H, W, lab = to_dev_bf16(b.H_bits), to_dev_bf16(b.W_bits), torch.from_numpy(b.labels).cuda()
    loss = torch.empty(w.T, dtype=torch.float32, device="cuda")
    lse = torch.empty_like(loss)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    prev = vp.vp_ce_set_wait_limit_ns(LIMIT_NS)
    try:
        vp.vp_ce_debug_drop_copy(0, 0, 1)
        vp.vp_ce_forward_static(H, W, lab, w.block_v, IGNORE_INDEX, loss, lse, w.T_chunk, 0, status)
        torch.cuda.synchronize()
    finally:
        vp.vp_ce_debug_drop_copy(-1)
        vp.vp_ce_set_wait_limit_ns(prev)
    assert int(status.item()) & WAIT_EXPIRED
    vp.vp_ce_forward_static(H, W, lab, w.block_v, IGNORE_INDEX, loss, lse, w.T_chunk, 0, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.abs(lse.cpu().numpy() - ref["lse"]).max() <= TOL_TOKEN


def test_an_armed_hook_for_another_kernel_kind_leaves_a_call_alone():
    w, b, ref = _problem(pair=True)
    run = DeviceRun(b.H_bits, b.W_bits, b.labels, w.block_v, w.T_chunk)
    try:
        vp.vp_ce_debug_drop_copy(3, 0, 1)          # weight-gradient GEMM: the forward does not launch one
        run.forward()
    finally:
        vp.vp_ce_debug_drop_copy(-1)
    assert run.fwd_status == 0
    assert np.abs(run.np_lse() - ref["lse"]).max() <= TOL_TOKEN
