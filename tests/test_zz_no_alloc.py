"""vp_ce_forward_static: the forward for callers that may not allocate device memory (plug-ins
living inside another runtime's memory plan, serving loops that must not synchronise on an
allocation).  Its scratch is a fixed array inside the library, so this test checks the two things
such a caller relies on: the results equal those of vp_ce_forward, and a second call that finds
the first call's leftovers in the shared array is still right.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import paper_2609_14306_b200 as vp
from synth_inputs import IGNORE_INDEX, custom_workload, make_batch
from vpce_testlib import TOL_TOKEN, to_dev_bf16

pytestmark = pytest.mark.gpu


def _inputs(seed, T, d, V, ignore_frac):
    w = custom_workload("noalloc", T=T, d=d, V=V, block_v=512, T_chunk=256, w_std=1.0 / np.sqrt(d),
                        labels="zipf", ignore_frac=ignore_frac, seed=seed)
    b = make_batch(w)
    return w, to_dev_bf16(b.H_bits), to_dev_bf16(b.W_bits), torch.from_numpy(b.labels).cuda()


def test_static_scratch_forward_matches_workspace_forward_twice():
    # two calls in a row with different shapes and data: the second finds the first one's state in the array
    for seed, T, d, V, frac in [(101, 600, 256, 3000, 0.1), (202, 384, 320, 1800, 0.0)]:
        w, H, W, lab = _inputs(seed, T, d, V, frac)
        ws = torch.empty(vp.vp_ce_workspace_bytes(w.T_chunk, w.d, w.block_v), dtype=torch.uint8, device="cuda")
        loss_ref = torch.empty(T, dtype=torch.float32, device="cuda")
        lse_ref = torch.empty_like(loss_ref)
        vp.vp_ce_forward(H, W, lab, w.block_v, IGNORE_INDEX, loss_ref, lse_ref, w.T_chunk, 2, ws)
        loss = torch.full_like(loss_ref, float("nan"))
        lse = torch.full_like(loss_ref, float("nan"))
        status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        vp.vp_ce_forward_static(H, W, lab, w.block_v, IGNORE_INDEX, loss, lse, w.T_chunk, 2, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.isfinite(lse).all() and torch.isfinite(loss).all()
        assert float((lse - lse_ref).abs().max()) <= TOL_TOKEN
        assert float((loss - loss_ref).abs().max()) <= TOL_TOKEN
        # same kernels, same order: in fact bit-identical
        assert torch.equal(lse, lse_ref) and torch.equal(loss, loss_ref)


def test_static_scratch_rejects_sizes_beyond_its_array():
    w, H, W, lab = _inputs(303, 256, 128, 1024, 0.0)
    loss = torch.empty(w.T, dtype=torch.float32, device="cuda")
    lse = torch.empty_like(loss)
    with pytest.raises(vp.VpceError) as ei:
        vp.vp_ce_forward_static(H, W, lab, 32768, IGNORE_INDEX, loss, lse, 16384, 0)
    assert ei.value.code == 5
    assert "scratch" in vp.vp_ce_status_string(5)
