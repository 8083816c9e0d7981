"""Property tests of the oracle on random small shapes (hypothesis): the Algorithm 3 restatement equals the
dense definition for any shard width, chunk size and rotation, and the gradients keep their invariants."""
import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import vpce_oracle as orc

IGN = -100


@st.composite
def problems(draw):
    T = draw(st.integers(1, 12))
    d = draw(st.integers(1, 6))
    V = draw(st.integers(1, 20))
    seed = draw(st.integers(0, 2 ** 16))
    rng = np.random.default_rng(seed)
    H = rng.standard_normal((T, d)) * draw(st.sampled_from([0.1, 1.0, 5.0]))
    W = rng.standard_normal((V, d))
    lab = rng.integers(0, V, size=T).astype(np.int32)
    lab[rng.random(T) < 0.2] = IGN
    return H, W, lab, draw(st.integers(1, 25)), draw(st.integers(1, 13)), draw(st.integers(0, 7))


@settings(max_examples=60, deadline=None)
@given(problems())
def test_ring_equals_dense_everywhere(prob):
    H, W, lab, block_v, T_chunk, base = prob
    lse, loss = orc.dense_forward(H, W, lab, IGN)
    l2, s2, gathers = orc.ring_fold_forward(H, W, lab, block_v, T_chunk, base, IGN)
    np.testing.assert_allclose(l2, lse, rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(s2, loss, rtol=1e-10, atol=1e-11)
    assert np.array_equal(gathers, (lab != IGN).astype(np.int64))
    dH, dW = orc.dense_backward(H, W, lab, None, IGN)
    rH, rW = orc.ring_backward(H, W, lab, lse, block_v, T_chunk, base, None, IGN)
    np.testing.assert_allclose(rH, dH, atol=1e-11)
    np.testing.assert_allclose(rW, dW, atol=1e-11)
    # every residual row sums to zero, ignored tokens get no gradient, the loss is non-negative
    np.testing.assert_allclose(dW.sum(0), 0.0, atol=1e-11)
    assert not dH[lab == IGN].any()
    assert (loss >= -1e-12).all()
