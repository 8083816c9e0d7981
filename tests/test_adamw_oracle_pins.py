"""Pins of the AdamW oracle against what mathematics and a library fix: a hand-worked step, closed forms,
torch.optim.AdamW in float64 over several steps, bf16 rounding against torch, bucket invariance."""
import numpy as np
import pytest
import torch

from oracle import adamw_oracle as ao

HP = dict(lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)


def test_hand_worked_first_step():
    # p = 1, g = 0.5, zero moments, t = 1, lr = 0.1, wd = 0.5, beta1 = 0.5, beta2 = 0.75, eps = 0:
    # decay: p = 1 * (1 - 0.05) = 0.95;  m = 0.25, v = 0.0625;  m_hat = 0.25 / 0.5 = 0.5;  v_hat = 0.0625 / 0.25 = 0.25
    # update: 0.95 - 0.1 * 0.5 / 0.5 = 0.85
    p, m, v, _ = ao.adamw_step(np.array([1.0]), np.array([0.0]), np.array([0.0]), np.array([0.5]), 1, 0.1, 0.5, 0.75,
                               0.0, 0.5)
    assert p[0] == pytest.approx(0.85, abs=1e-15) and m[0] == 0.25 and v[0] == 0.0625
    # second step with g = -1: decay 0.85 * 0.95 = 0.8075; m = 0.125 - 0.5 = -0.375; v = 0.046875 + 0.25 = 0.296875
    # m_hat = -0.375 / 0.75 = -0.5; v_hat = 0.296875 / 0.4375 = 0.678571428...; sqrt = 0.823754471...
    p2, m2, v2, _ = ao.adamw_step(p, m, v, np.array([-1.0]), 2, 0.1, 0.5, 0.75, 0.0, 0.5)
    assert m2[0] == -0.375 and v2[0] == 0.296875
    assert p2[0] == pytest.approx(0.8075 + 0.1 * 0.5 / np.sqrt(0.296875 / 0.4375), abs=1e-15)


def test_closed_forms():
    rng = np.random.default_rng(0)
    n = 1000
    p, g = rng.standard_normal(n), rng.standard_normal(n)
    z = np.zeros(n)
    # t = 1 from zero moments: m_hat = g, v_hat = g^2, so the step is lr * g / (|g| + eps): lr * sign(g) up to eps
    p1, _, _, _ = ao.adamw_step(p, z, z, g, 1, 1e-3, 0.9, 0.999, 1e-12, 0.0)
    np.testing.assert_allclose(p1, p - 1e-3 * g / (np.abs(g) + 1e-12), rtol=0, atol=1e-15)
    np.testing.assert_allclose(p1, p - 1e-3 * np.sign(g), rtol=0, atol=2e-3 * 1e-12 / np.abs(g).min())
    # lr = 0: the parameter does not move, the moments still do
    p2, m2, v2, _ = ao.adamw_step(p, z, z, g, 3, 0.0, 0.9, 0.999, 1e-8, 0.1)
    np.testing.assert_array_equal(p2, p)
    np.testing.assert_allclose(m2, 0.1 * g, rtol=1e-15)
    np.testing.assert_allclose(v2, 0.001 * g * g, rtol=1e-12)
    # g = 0 and zero moments: pure decoupled decay
    p3, m3, v3, _ = ao.adamw_step(p, z, z, z, 5, 1e-2, 0.9, 0.999, 1e-8, 0.1)
    np.testing.assert_allclose(p3, p * (1 - 1e-3), rtol=1e-15)
    assert not m3.any() and not v3.any()
    # weight_decay = 0 is Adam: the sign of the step follows the first moment
    p4, m4, _, _ = ao.adamw_step(p, 0.3 * g, np.abs(g), g, 7, 1e-2, 0.9, 0.999, 1e-8, 0.0)
    assert np.all(np.sign(p - p4) == np.sign(m4))
    with pytest.raises(ValueError):
        ao.adamw_step(p, z, z, g, 0, 1e-3, 0.9, 0.999, 1e-8, 0.0)


def test_matches_torch_adamw_float64_over_steps():
    rng = np.random.default_rng(1)
    n = 4096
    p0 = rng.standard_normal(n).astype(np.float32).astype(np.float64)
    tp = torch.nn.Parameter(torch.from_numpy(p0.copy()))
    opt = torch.optim.AdamW([tp], lr=HP["lr"], betas=(HP["beta1"], HP["beta2"]), eps=HP["eps"],
                            weight_decay=HP["weight_decay"])
    p, m, v = p0.copy(), np.zeros(n), np.zeros(n)
    for step in range(1, 6):
        g = rng.standard_normal(n) * (0.1 if step % 2 else 3.0)
        tp.grad = torch.from_numpy(g.copy())
        opt.step()
        p, m, v, _ = ao.adamw_step(p, m, v, g, step, **HP)
        np.testing.assert_allclose(p, tp.detach().numpy(), rtol=1e-12, atol=1e-14)
        st = opt.state[tp]
        np.testing.assert_allclose(m, st["exp_avg"].numpy(), rtol=1e-12, atol=1e-16)
        np.testing.assert_allclose(v, st["exp_avg_sq"].numpy(), rtol=1e-12, atol=1e-16)


def test_bf16_rounding_is_nearest_even():
    rng = np.random.default_rng(2)
    x = np.concatenate([rng.standard_normal(100000).astype(np.float32) * 10.0 ** rng.integers(-6, 6, 100000),
                        np.array([1.00390625, 1.01171875, 0.0, -0.0, 3.0e38, 1e-40], dtype=np.float32)])
    # 1.00390625 = 1 + 2^-8 lies half way between 1 and 1 + 2^-7: ties go to the even mantissa (1.0);
    # 1.01171875 = 1 + 3 * 2^-8 lies half way between 1 + 2^-7 and 1 + 2^-6: even is 1 + 2^-6
    bits = ao.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, ref)
    assert bits[100000] == 0x3F80 and bits[100001] == 0x3F82
    _, _, _, w = ao.adamw_step(x, np.zeros_like(x), np.zeros_like(x), np.zeros_like(x), 1, 0.0, 0.9, 0.999, 1e-8, 0.0)
    np.testing.assert_array_equal(w, bits)                   # the working weight is the rounding of the new master


@pytest.mark.parametrize("bucket", [1, 7, 100, 1000, 5000])
def test_bucketing_changes_nothing(bucket):
    rng = np.random.default_rng(3)
    n = 1000
    p, m, v, g = (rng.standard_normal(n) for _ in range(4))
    v = np.abs(v)
    whole = ao.adamw_step(p, m, v, g, 4, **HP)
    parts = ao.streamed_step(p, m, v, g, 4, bucket_params=bucket, **HP)
    for a, b in zip(whole, parts):
        np.testing.assert_array_equal(a, b)
    uneven = ao.streamed_step(p, m, v, g, 4, bucket_params=0, offsets=[0, 3, 500, 999, 1000], **HP)
    for a, b in zip(whole, uneven):
        np.testing.assert_array_equal(a, b)
    assert ao.bucket_ranges(10, 4) == [(0, 4), (4, 8), (8, 10)]
    with pytest.raises(ValueError):
        ao.bucket_ranges(10, 4, offsets=[0, 5, 5, 10])
