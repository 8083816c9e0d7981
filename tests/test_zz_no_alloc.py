"""vp_ce_forward_static: the forward for callers that may not allocate device memory (plug-ins
living inside another runtime's memory plan, serving loops that must not synchronise on an
allocation).  Its scratch is a fixed array inside the library, so this test checks what such a
caller relies on: the results are those of the float64 oracle and of vp_ce_forward; a second call
that finds the first call's leftovers in the shared array is still right; the call really takes no
device memory; and the documented size limit is enforced.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import paper_2609_14306_b200 as vp
from oracle import vpce_oracle as orc
from synth_inputs import IGNORE_INDEX, bf16_bits_to_f64, custom_workload, make_batch
from vpce_testlib import TOL_MEAN_REL, TOL_TOKEN, to_dev_bf16

pytestmark = pytest.mark.gpu


def _inputs(seed, T, d, V, ignore_frac, block_v=512, T_chunk=256):
    w = custom_workload("noalloc", T=T, d=d, V=V, block_v=block_v, T_chunk=T_chunk, w_std=1.0 / np.sqrt(d),
                        labels="zipf", ignore_frac=ignore_frac, seed=seed)
    b = make_batch(w)
    return w, b, to_dev_bf16(b.H_bits), to_dev_bf16(b.W_bits), torch.from_numpy(b.labels).cuda()


def _static_forward(w, H, W, lab, base):
    loss = torch.full((w.T,), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full_like(loss, float("nan"))
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    vp.vp_ce_forward_static(H, W, lab, w.block_v, IGNORE_INDEX, loss, lse, w.T_chunk, base, status)
    torch.cuda.synchronize()
    return loss, lse, int(status.item())


def _check_against_oracle(w, b, loss, lse):
    lse_ref, loss_ref = orc.dense_forward(bf16_bits_to_f64(b.H_bits), bf16_bits_to_f64(b.W_bits), b.labels, IGNORE_INDEX)
    assert np.abs(lse.cpu().numpy().astype(np.float64) - lse_ref).max() <= TOL_TOKEN
    assert np.abs(loss.cpu().numpy().astype(np.float64) - loss_ref).max() <= TOL_TOKEN
    mean_ref, n_valid = orc.masked_mean(loss_ref, b.labels, IGNORE_INDEX)
    if n_valid:
        mean = float(loss.double()[torch.from_numpy(b.labels != IGNORE_INDEX).cuda()].mean())
        assert abs(mean - mean_ref) <= TOL_MEAN_REL * abs(mean_ref)


def test_static_scratch_forward_matches_oracle_and_workspace_forward_twice():
    # two calls in a row with different shapes and data: the second finds the first one's state in the array
    for seed, T, d, V, frac in [(101, 600, 256, 3000, 0.1), (202, 384, 320, 1800, 0.0)]:
        w, b, H, W, lab = _inputs(seed, T, d, V, frac)
        loss, lse, status = _static_forward(w, H, W, lab, base=2)
        assert status == 0
        assert torch.isfinite(lse).all() and torch.isfinite(loss).all()
        _check_against_oracle(w, b, loss, lse)
        # and the entry point with a caller workspace: same kernels, same order, hence bit-identical
        ws = torch.empty(vp.vp_ce_workspace_bytes(w.T_chunk, w.d, w.block_v), dtype=torch.uint8, device="cuda")
        loss_ws = torch.empty(T, dtype=torch.float32, device="cuda")
        lse_ws = torch.empty_like(loss_ws)
        vp.vp_ce_forward(H, W, lab, w.block_v, IGNORE_INDEX, loss_ws, lse_ws, w.T_chunk, 2, ws)
        torch.cuda.synchronize()
        assert torch.equal(lse, lse_ws) and torch.equal(loss, loss_ws)


def test_static_scratch_at_its_documented_maximum():
    # T_chunk = 4096 with block_v = 8192 is the size the header promises; the vocabulary ends inside a tile
    w, b, H, W, lab = _inputs(404, 4096 + 130, 64, 8192 + 300, 0.05, block_v=8192, T_chunk=4096)
    loss, lse, status = _static_forward(w, H, W, lab, base=1)
    assert status == 0
    _check_against_oracle(w, b, loss, lse)


def test_static_scratch_call_takes_no_device_memory():
    w, b, H, W, lab = _inputs(505, 512, 128, 2048, 0.0)
    loss, lse, _ = _static_forward(w, H, W, lab, base=0)          # first call: module load, address look-up
    vp.vp_ce_profile_enable(True)                                  # the event-recording path must not be taken either
    try:
        status = torch.zeros(1, dtype=torch.int32, device="cuda")      # allocated before the measured window
        # what earlier tests left behind (tensors, a captured graph's pool) is released now, not inside the window
        import gc
        gc.collect()
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        vp.vp_ce_forward_static(H, W, lab, w.block_v, IGNORE_INDEX, loss, lse, w.T_chunk, 0, status)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
        assert free1 >= free0, (free0, free1)                      # the driver handed out nothing either
    finally:
        vp.vp_ce_profile_enable(False)
    assert all(n == 0 for _, n in vp.vp_ce_profile_collect().values())
    _check_against_oracle(w, b, loss, lse)


def test_static_scratch_rejects_sizes_beyond_its_array():
    w, b, H, W, lab = _inputs(303, 256, 128, 1024, 0.0)
    loss = torch.empty(w.T, dtype=torch.float32, device="cuda")
    lse = torch.empty_like(loss)
    n0 = vp.vp_ce_launch_count()
    # far beyond the array, and the first token chunk (a multiple of 128) whose layout no longer fits at block_v = 8192
    for block_v, T_chunk in [(32768, 16384), (8192, 4992)]:
        with pytest.raises(vp.VpceError) as ei:
            vp.vp_ce_forward_static(H, W, lab, block_v, IGNORE_INDEX, loss, lse, T_chunk, 0)
        assert ei.value.code == 5
    assert vp.vp_ce_launch_count() == n0                            # a rejected call launches nothing
    assert "scratch" in vp.vp_ce_status_string(5)
