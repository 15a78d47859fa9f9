"""GPU parity for the scaled Rand-k compressor (Appendix, Lemma 8 and Example 2) inside Algorithm 2: bit for bit against
the oracle on supplied gradients, iteration by iteration on the logistic objective; the index sets are inputs drawn
by ef21_inputs.randk_sets for both sides."""
import numpy as np
import pytest
import torch

import ef21_inputs as inputs
import oracle as oracle_mod
from gpu_util import assert_state_bitwise, dev, make_gpu, make_oracle_state, rel_l2, set_gpu_state_from_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2106_05203_b200 import binding
    return binding


@pytest.mark.parametrize("n,d,k", [(2, 4, 1), (5, 300, 7), (3, 5000, 50), (8, 70001, 700), (4, 300000, 300), (6, 64, 64)])
def test_supplied_gradients_randk_bit_exact(n, d, k, B, oracle32):
    rng = np.random.default_rng(d + k)
    steps = 6
    sets = inputs.randk_sets(d, steps, n, d, k)
    h = B.EF21(n, d, k, 0.05); st = oracle_mod.State(oracle32, n, d, k, 0.05)
    h.init_grads(None, B.INIT_ZERO); st.init(1)
    for t in range(steps):                       # changing gradients, one call per step
        V = rng.standard_normal((n, d)).astype(np.float32)
        h.step_randk(dev(sets[t:t + 1], torch.int32), dev(V)); st.step_randk(sets[t:t + 1], V)
        assert_state_bitwise(h, st, f"step {t}")
    V = rng.standard_normal((n, d)).astype(np.float32)
    h.step_randk(dev(sets, torch.int32), dev(V)); st.step_randk(sets, V)      # static input, all steps in one call
    assert_state_bitwise(h, st, "six steps in one call")
    assert h.poll() == 0


@pytest.mark.parametrize("cfg,k,steps", [(0, 4, 40), (1, 1, 60), (2, 16, 25), (3, 8, 10)])
def test_logistic_randk_tracks_the_oracle(cfg, k, steps, B, oracle32):
    # no selection by magnitude, hence no near-ties: the same coordinates on both sides, values within the gradient tolerance
    w = inputs.config(cfg, k=k)
    sets = inputs.randk_sets(7 + cfg, steps, w.n, w.d, k)
    h = make_gpu(w, k=k); st = make_oracle_state(oracle32, w, k=k)
    h.init(B.INIT_ZERO); st.init(1)
    for t in range(steps):
        h.step_randk(dev(sets[t:t + 1], torch.int32)); st.step_randk(sets[t:t + 1])
        x, g, gi, li, lv = h.get_state_host()
        np.testing.assert_array_equal(li, sets[t])
        np.testing.assert_array_equal(li, st.idx)
        scale = np.max(np.abs(st.grads()), axis=1, keepdims=True)
        assert np.all(np.abs(lv.astype(np.float64) - st.val) <= 1e-5 * scale), t
        assert rel_l2(x, st.x) <= 1e-4 or np.linalg.norm(st.x) == 0
        set_gpu_state_from_oracle(h, st)
    # free-running, all steps in one call
    h2 = make_gpu(w, k=k); st2 = make_oracle_state(oracle32, w, k=k)
    h2.init(B.INIT_ZERO); st2.init(1)
    h2.step_randk(dev(sets, torch.int32)); st2.step_randk(sets)
    assert rel_l2(h2.get_state_host()[0], st2.x) <= 1e-4
    assert h2.eval()[0] == pytest.approx(st2.loss(), rel=1e-4)
    assert h.poll() == 0 and h2.poll() == 0


def test_randk_bad_sets_are_reported(B):
    n, d, k = 3, 100, 4
    h = B.EF21(n, d, k, 0.1); h.init_grads(None, B.INIT_ZERO)
    V = dev(np.ones((n, d), dtype=np.float32))
    good = inputs.randk_sets(1, 1, n, d, k)
    h.step_randk(dev(good, torch.int32), V)
    assert h.poll() == 0
    for bad_value, pos in ((d, 3), (-1, 0), (None, 2)):
        bad = good.copy()
        bad[0, 1, pos] = bad[0, 1, pos - 1] if bad_value is None else bad_value       # repeated / out of range
        h.step_randk(dev(bad, torch.int32), V)
        assert h.poll() == 1
        h.clear_status()
    h.step_randk(dev(good, torch.int32), V)
    assert h.poll() == 0
