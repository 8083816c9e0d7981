"""GPU parity of the bucket-streamed AdamW (fused update kernel and the three-stream bucket pipeline) against the
float64 oracle on the same seeded fp32 state.

Tolerances (fp32 arithmetic against float64, stated per quantity): every kernel operation is a correctly rounded
fp32 operation, so each result carries a few units of 2^-24 relative to the LARGEST term that entered it:
  m: 4e-7 (|m_old| + |g|)        v: 4e-7 (v_old + g^2)
  p: 2.5e-7 |p_old| + 4e-6 |step taken| (the quotient m / (sqrt(v) + eps) goes through four roundings)
     + the bound on m's error carried through lr / (1 - beta1^t) / (sqrt(v_hat) + eps) (m may cancel)
The bf16 working weight is a rounding decision taken on the fp32 master: it must equal the nearest-even rounding of
the GPU's own new master bit for bit (a property), and equal the oracle's rounding except where the two fp32 masters
straddle a rounding boundary (at most a 1e-3 fraction of the elements); every working weight lies within half a
bf16 step (plus the master's tolerance) of the oracle's float64 master."""
import numpy as np
import pytest
import torch

import paper_2609_14306_b200 as vp
from oracle import adamw_oracle as ao

pytestmark = pytest.mark.gpu

HP = dict(lr=3e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)


def _state(n, seed):
    rng = np.random.default_rng(seed)
    p = (rng.standard_normal(n) * 0.05).astype(np.float32)
    m = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    v = (rng.standard_normal(n) ** 2 * 1e-6).astype(np.float32)
    g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-5, -1, n)).astype(np.float32)
    g[::97] = 0.0                                           # exact zeros: the eps branch of the denominator
    return p, m, v, g


def _check(p_old, m_old, v_old, g, got, step, hp=HP):
    p_ref, m_ref, v_ref, w_ref = ao.adamw_step(p_old, m_old, v_old, g, step, **hp)
    p, m, v, w_bits = got
    p64, m64, v64 = p.astype(np.float64), m.astype(np.float64), v.astype(np.float64)
    a = lambda x: np.abs(x.astype(np.float64))
    assert np.all(np.abs(m64 - m_ref) <= 4e-7 * (a(m_old) + a(g)) + 1e-38)
    assert np.all(np.abs(v64 - v_ref) <= 4e-7 * (a(v_old) + a(g) ** 2) + 1e-38)
    taken = np.abs(p_ref - p_old.astype(np.float64) * (1.0 - hp["lr"] * hp["weight_decay"]))
    # the first moment may cancel (beta1 m and (1 - beta1) g of opposite sign): its ABSOLUTE error, bounded above,
    # then enters the step divided by the denominator
    denom = np.sqrt(v_ref / (1.0 - hp["beta2"] ** step)) + hp["eps"]
    from_m = hp["lr"] / (1.0 - hp["beta1"] ** step) * 4e-7 * (a(m_old) + a(g)) / denom
    tol_p = 2.5e-7 * a(p_old) + 4e-6 * taken + from_m + 1e-38
    assert np.all(np.abs(p64 - p_ref) <= tol_p)
    np.testing.assert_array_equal(w_bits, ao.f32_to_bf16_bits(p))              # w = bf16(new master), bit for bit
    diff = w_bits != w_ref
    assert diff.mean() <= 1e-3                                                 # the oracle's rounding, except ...
    # ... where the two masters straddle a rounding boundary: the GPU's working weight is still a correct rounding of
    # the true value up to the master's own tolerance (half a bf16 step of its magnitude: 2^(exponent - 8))
    w_val = (w_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    half_step = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(w_val), 1e-300))) - 8)
    assert np.all(np.abs(w_val - p_ref) <= half_step + tol_p)
    return p_ref, m_ref, v_ref


def _bits(w):
    return w.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("n", [1, 3, 4, 1027, (1 << 20) + 3])
def test_fused_update_kernel_matches_oracle_over_steps(n):
    p, m, v, g = _state(n, seed=n)
    dp, dm, dv = (torch.from_numpy(x.copy()).cuda() for x in (p, m, v))
    w = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    for step in (1, 2, 7):
        g = np.roll(g, step)
        dg = torch.from_numpy(g.copy()).cuda()
        vp.osadamw_update_device(dp, dm, dv, dg, w, step=step, **HP)
        torch.cuda.synchronize()
        got = (dp.cpu().numpy(), dm.cpu().numpy(), dv.cpu().numpy(), _bits(w))
        _check(p, m, v, g, got, step)
        p, m, v = got[0].copy(), got[1].copy(), got[2].copy()                  # next step starts from the fp32 state


def test_update_kernel_special_cases():
    n = 4096
    p, m, v, g = _state(n, seed=5)
    z = np.zeros(n, dtype=np.float32)
    dp, dm, dv, dg = (torch.from_numpy(x.copy()).cuda() for x in (p, z, z, g))
    w = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    # lr = 0: the master does not move at all, the moments do
    vp.osadamw_update_device(dp, dm, dv, dg, w, 0.0, 0.9, 0.999, 1e-8, 0.1, 1)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(dp.cpu().numpy(), p)
    np.testing.assert_allclose(dm.cpu().numpy(), 0.1 * g.astype(np.float64), rtol=3e-7, atol=0)
    # t = 1 from zero moments, no decay: a step of lr * sign(g) (up to eps), 0 where g = 0
    dp, dm, dv = (torch.from_numpy(x.copy()).cuda() for x in (p, z, z))
    vp.osadamw_update_device(dp, dm, dv, dg, w, 1e-3, 0.9, 0.999, 1e-12, 0.0, 1)
    torch.cuda.synchronize()
    big = np.abs(g) > 1e-4
    np.testing.assert_allclose((dp.cpu().numpy().astype(np.float64) - p)[big], -1e-3 * np.sign(g)[big], rtol=1e-4, atol=1e-9)
    assert not (dp.cpu().numpy() - p)[g == 0].any()
    for bad in (dict(step=0), dict(beta1=1.0), dict(eps=-1.0)):
        kw = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, step=1)
        kw.update(bad)
        with pytest.raises(vp.VpceError) as ei:
            vp.osadamw_update_device(dp, dm, dv, dg, w, **kw)
        assert ei.value.code == 1


def _pinned(x):
    return torch.from_numpy(x.copy()).pin_memory()


@pytest.mark.parametrize("bucket,slots,offsets", [
    (100_000, 2, None),            # 11 buckets, the last one short; 2 slots (the paper's chosen depth)
    (262_144, 3, None),
    (1 << 21, 2, None),            # one bucket holds everything
    (400_000, 2, [0, 4, 300_000, 300_004, 700_000, 1_048_584]),     # caller-defined bucket boundaries
])
def test_bucket_pipeline_matches_oracle_and_is_bucket_invariant(bucket, slots, offsets):
    n = (1 << 20) + 8
    p, m, v, g = _state(n, seed=11)
    hp, hm, hv = _pinned(p), _pinned(m), _pinned(v)
    w = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    staging = torch.empty(vp.osadamw_staging_bytes(bucket, slots), dtype=torch.uint8, device="cuda")
    h = vp.osadamw_create(bucket, slots, staging)
    try:
        for step in (1, 2, 3):
            g = np.roll(g, 17 * step)
            hg = _pinned(g)
            p_old, m_old, v_old = hp.numpy().copy(), hm.numpy().copy(), hv.numpy().copy()
            vp.osadamw_step(h, hp, hm, hv, hg, w, step=step, bucket_offsets=offsets, **HP)
            w_seen = w.float().sum()                          # enqueued right behind the step on the caller's stream
            vp.osadamw_wait(h)
            got = (hp.numpy().copy(), hm.numpy().copy(), hv.numpy().copy(), _bits(w))
            _check(p_old, m_old, v_old, g, got, step)
            assert float(w_seen) == float(w.float().sum())    # the caller's stream was ordered behind the last update
            # bucketing changes nothing: the same step by the plain kernel on the whole shard gives the same bits
            dp, dm, dv, dg = (torch.from_numpy(x.copy()).cuda() for x in (p_old, m_old, v_old, g))
            w2 = torch.zeros_like(w)
            vp.osadamw_update_device(dp, dm, dv, dg, w2, step=step, **HP)
            torch.cuda.synchronize()
            np.testing.assert_array_equal(dp.cpu().numpy(), got[0])
            np.testing.assert_array_equal(dm.cpu().numpy(), got[1])
            np.testing.assert_array_equal(dv.cpu().numpy(), got[2])
            assert torch.equal(w2.view(torch.int16), w.view(torch.int16))
    finally:
        vp.osadamw_destroy(h)


def test_pipeline_argument_checks():
    n = 1000
    p, m, v, g = _state(n, seed=3)
    hp, hm, hv, hg = _pinned(p), _pinned(m), _pinned(v), _pinned(g)
    w = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    staging = torch.empty(vp.osadamw_staging_bytes(256, 2), dtype=torch.uint8, device="cuda")
    with pytest.raises(vp.VpceError) as ei:
        vp.osadamw_create(512, 2, staging)                    # staging of a smaller pipeline
    assert ei.value.code == 3
    h = vp.osadamw_create(256, 2, staging)
    try:
        with pytest.raises(vp.VpceError) as ei:               # a caller-defined bucket longer than the slots
            vp.osadamw_step(h, hp, hm, hv, hg, w, step=1, bucket_offsets=[0, 400, 1000], **HP)
        assert ei.value.code == 1
        with pytest.raises(vp.VpceError) as ei:
            vp.osadamw_step(h, hp, hm, hv, hg, w, step=0, **HP)
        assert ei.value.code == 1
        vp.osadamw_step(h, hp, hm, hv, hg, w, step=1, **HP)   # and a valid call still works afterwards
        vp.osadamw_wait(h)
        _check(p, m, v, g, (hp.numpy(), hm.numpy(), hv.numpy(), _bits(w)), 1)
    finally:
        vp.osadamw_destroy(h)
