"""GPU parity for the least-squares objective (Appendix A.2): gradients, evaluation and EF21
trajectories on both execution paths against the oracle."""
import numpy as np
import pytest

import ef21_inputs as inputs
import oracle as oracle_mod
from gpu_util import dev, lockstep, make_gpu, make_oracle_state, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2106_05203_b200 import binding
    return binding


@pytest.fixture
def ls32(oracle32):
    oracle32.set_objective(1)
    yield oracle32
    oracle32.set_objective(0)


def _ls_workload(cfg):
    w = inputs.config(cfg)
    w.lam = 0.0
    w.gamma = inputs.gamma_one_over_L(w.A, w.row_offsets, 0.0, "least_squares")
    return w


@pytest.mark.parametrize("cfg", [0, 1, 3])
def test_least_squares_gradients(cfg, B, ls32):
    w = _ls_workload(cfg)
    h = make_gpu(w); h.set_objective(B.OBJECTIVE_LEAST_SQUARES)
    x = (np.random.default_rng(cfg).standard_normal(w.d) * 0.2).astype(np.float32)
    h.set_x(dev(x))
    got = h.local_grads().cpu().numpy()
    want = ls32.all_grads(w.A, w.y, w.row_offsets, x, w.lam)
    for i in range(w.n):
        assert rel_l2(got[i], want[i]) <= 1e-5
    h.init(1)
    assert h.eval()[0] == pytest.approx(ls32.loss(w.A, w.y, w.row_offsets, x, w.lam), rel=1e-5)


@pytest.mark.parametrize("path", [1, 2], ids=["launches", "persistent"])
@pytest.mark.parametrize("cfg,k,steps", [(0, 4, 40), (1, 1, 60), (2, 4, 20)])
def test_least_squares_lockstep(cfg, k, steps, path, B, ls32):
    w = _ls_workload(cfg)
    h = make_gpu(w, k=k, path=path); h.set_objective(B.OBJECTIVE_LEAST_SQUARES)
    st = make_oracle_state(ls32, w, k=k)
    h.init(0); st.init(0)
    assert lockstep(h, st, ls32, w, steps, k=k) <= max(2, steps // 10)
    assert h.last_path == path
    x = h.get_state_host()[0]
    assert rel_l2(x, st.x) <= 1e-4
    assert h.eval()[0] == pytest.approx(st.loss(), rel=1e-4)
