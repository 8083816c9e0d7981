"""The K-split tail of the gradient GEMMs: when the output tiles do not fill whole rounds of the CTA pairs, the
remainder tiles run as several parts along the contracted dimension, and the parts of a tile add into the output in
the order of their index (flags in the workspace).  The library decides per geometry whether to split; these tests
force the split (vp_ce_set_tail_parts) on shapes the float64 oracle can check element by element, with and without
staggered part lengths, with the narrow last column tile, across shards (the input gradient accumulates) and across
chunks (the weight gradient accumulates), and check that the result is bitwise reproducible and that a lost copy
inside a split tile ends in the give-up path like any other."""
import time

import numpy as np
import pytest
import torch

import paper_2609_14306_b200 as vp
from oracle import vpce_oracle as orc
from synth_inputs import IGNORE_INDEX, bf16_bits_to_f64, custom_workload, make_batch
from vpce_testlib import TOL_GRAD, TOL_TOKEN, DeviceRun, check_against_oracle, relF

pytestmark = pytest.mark.gpu


@pytest.fixture
def tail_parts():
    prev = vp.vp_ce_set_tail_parts(-1)
    yield vp.vp_ce_set_tail_parts
    vp.vp_ce_set_tail_parts(prev)


def _run(w, b, base=0):
    return DeviceRun(b.H_bits, b.W_bits, b.labels, w.block_v, w.T_chunk, base).forward().backward()


@pytest.mark.parametrize("parts", [2, 3, 5])
@pytest.mark.parametrize("T,d,V,block_v,T_chunk", [
    (4096, 320, 4096, 2048, 2048),   # 32 k-blocks in both gradient GEMMs (staggered parts fit at 2), 2 shards x 2 chunks,
                                     # last column tile 64 wide
    (1024, 512, 1536, 512, 512),     # 8 k-blocks: equal parts; three shards, two chunks
    (896, 256, 2304, 768, 384),      # token chunk of three 128-row tiles: the pair's last tile is half padding
])
def test_forced_split_matches_oracle_and_is_reproducible(tail_parts, parts, T, d, V, block_v, T_chunk):
    w = custom_workload(f"tail{T}x{d}", T=T, d=d, V=V, block_v=block_v, T_chunk=T_chunk, w_std=1.0 / np.sqrt(d),
                        labels="zipf", ignore_frac=0.05, seed=T + d + parts)
    b = make_batch(w)
    H64, W64 = bf16_bits_to_f64(b.H_bits), bf16_bits_to_f64(b.W_bits)
    ref = orc.forward_backward(H64, W64, b.labels, None, IGNORE_INDEX)
    tail_parts(0)
    whole = _run(w, b, base=1)
    tail_parts(parts)
    n0 = vp.vp_ce_launch_count()
    a = _run(w, b, base=1)
    c = _run(w, b, base=1)
    assert a.bwd_status == 0 and c.bwd_status == 0
    assert vp.vp_ce_launch_count() - n0 > 0
    e = check_against_oracle(a, ref, H64, W64, b.labels, orc.default_dloss(b.labels, IGNORE_INDEX), w.name)
    print(w.name, parts, {k: f"{v:.2e}" for k, v in e.items()})
    # one fixed summation order: run to run bitwise equal
    assert torch.equal(a.dW, c.dW) and torch.equal(a.dH.view(torch.int16), c.dH.view(torch.int16))
    # and the same sums as without the split up to the order of the additions
    assert relF(a.np_dW(), whole.np_dW()) <= 1e-5
    assert (a.dW != whole.dW).any(), "the split did not change the summation order: was it applied at all?"


@pytest.mark.parametrize("parts", [-1, 3])
def test_split_tail_is_bitwise_reproducible_at_the_benchmark_launch_geometry(tail_parts, parts):
    # the config-3 launch geometry (74 pairs, 384 / 768 tiles per gradient launch, 14 / 28 remainder tiles, narrow
    # last column tile), two shards; -1 is the library's own choice, which splits the weight-gradient launch here
    w = custom_workload("tailrep", T=16384, d=2880, V=16384, block_v=8192, T_chunk=16384, w_std=0.02,
                        labels="zipf", ignore_frac=0.05, seed=9)
    b = make_batch(w)
    tail_parts(0)
    whole = _run(w, b, base=1)
    tail_parts(parts)
    run = _run(w, b, base=1)
    assert run.bwd_status == 0
    dW0, dH0 = run.dW.clone(), run.dH.clone()
    assert (dW0 != whole.dW).any()                            # the split is in use
    assert relF(dW0.double().cpu().numpy(), whole.dW.double().cpu().numpy()) <= 1e-5
    for _ in range(10):
        run.dW.fill_(float("nan"))
        run.dH.fill_(float("nan"))
        run.backward()
        assert run.bwd_status == 0
        assert torch.equal(run.dW, dW0) and torch.equal(run.dH.view(torch.int16), dH0.view(torch.int16))


def test_lost_copy_inside_a_split_tile_gives_up_and_the_next_call_is_clean(tail_parts):
    w = custom_workload("tailgiveup", T=512, d=256, V=1024, block_v=512, T_chunk=256, w_std=0.0625,
                        labels="zipf", ignore_frac=0.05, seed=62)
    b = make_batch(w)
    ref = orc.forward_backward(bf16_bits_to_f64(b.H_bits), bf16_bits_to_f64(b.W_bits), b.labels)
    run = DeviceRun(b.H_bits, b.W_bits, b.labels, w.block_v, w.T_chunk).forward()
    tail_parts(2)
    prev = vp.vp_ce_set_wait_limit_ns(2_000_000)
    try:
        for kind in (2, 3):
            vp.vp_ce_debug_drop_copy(kind, 1, 3)          # k-block 1 of the first list entry: part 0 of a split tile
            t0 = time.perf_counter()
            run.backward()
            dt = time.perf_counter() - t0
            assert run.bwd_status & 2, (kind, run.bwd_status)
            assert dt < 1.0, dt
    finally:
        vp.vp_ce_debug_drop_copy(-1)
        vp.vp_ce_set_wait_limit_ns(prev)
    run.forward().backward()
    assert run.fwd_status == 0 and run.bwd_status == 0
    assert relF(run.np_dH(), ref["dH"]) <= TOL_GRAD and relF(run.np_dW(), ref["dW"]) <= TOL_GRAD
    assert np.abs(run.np_lse() - ref["lse"]).max() <= TOL_TOKEN
