"""GPU parity for the stochastic variant (Algorithm 5): minibatch gradient estimates over
caller-supplied rows and the EF21 trajectories built from them, against the oracle."""
import numpy as np
import pytest
import torch

import ef21_inputs as inputs
from gpu_util import assert_state_bitwise, dev, lockstep, make_gpu, make_oracle_state, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2106_05203_b200 import binding
    return binding


def _batch_grads(o, w, x, batch):
    out = np.empty((w.n, w.d), dtype=np.float64)
    for i in range(w.n):
        rows = w.row_offsets[i] + batch[i].astype(np.int64)
        out[i] = o.local_grad(w.A[rows], w.y[rows], x, w.lam)
    return out


@pytest.mark.parametrize("cfg,tau", [(0, 1), (0, 7), (1, 32), (1, 100), (3, 300), (3, 1000)])
def test_minibatch_estimates(cfg, tau, B, oracle32):
    # From g_i = 0, g = 0 and k = d the state after one iteration holds the estimates themselves.
    w = inputs.config(cfg)
    tau = min(tau, int(np.min(np.diff(w.row_offsets))))
    h = make_gpu(w, k=w.d); st = make_oracle_state(oracle32, w, k=w.d)
    h.init(1); st.init(1)
    batch = inputs.minibatch_rows(11, 0, w.row_offsets, tau)
    h.step_minibatch(dev(batch, torch.int32)); st.step_minibatch(batch)
    gi = h.get_state_host()[2]
    for i in range(w.n):
        assert rel_l2(gi[i], st.gi[i]) <= 1e-5, i
    assert h.poll() == 0


@pytest.mark.parametrize("path", [1, 2], ids=["launches", "persistent"])
@pytest.mark.parametrize("cfg,k,tau,steps", [(0, 4, 8, 40), (1, 1, 32, 60), (2, 4, 64, 25), (3, 8, 128, 10)])
def test_minibatch_lockstep(cfg, k, tau, steps, path, B, oracle32):
    w = inputs.config(cfg)
    h = make_gpu(w, k=k, path=path); st = make_oracle_state(oracle32, w, k=k)
    h.init(0); st.init(0)
    batches = {}

    def advance(t):
        batches[t] = inputs.minibatch_rows(5, t, w.row_offsets, tau)
        h.step_minibatch(dev(batches[t], torch.int32)); st.step_minibatch(batches[t])

    def grads_of(t):
        return _batch_grads(oracle32, w, st.x, batches[t])

    assert lockstep(h, st, oracle32, w, steps, k=k, advance=advance, grads_of=grads_of) <= max(2, steps // 10)
    assert h.last_path == path
    assert rel_l2(h.get_state_host()[0], st.x) <= 1e-4
    assert h.poll() == 0


@pytest.mark.parametrize("path", [0, 1], ids=["auto", "launches"])
@pytest.mark.parametrize("cfg,k,tau,steps", [(1, 1, 32, 80), (0, 4, 8, 30), (3, 1, 64, 12)])
def test_many_stochastic_iterations_in_one_call(cfg, k, tau, steps, path, B, oracle32):
    # [steps][n][tau] row numbers, one call (one launch of the persistent kernel on the automatic path): the same bits
    # as the same iterations one call each, and the oracle's trajectory
    w = inputs.config(cfg)
    all_rows = np.stack([inputs.minibatch_rows(9, t, w.row_offsets, tau) for t in range(steps)])
    outs = []
    for single in (False, True):
        h = make_gpu(w, k=k, path=path); h.init(0)
        if single:
            for t in range(steps):
                h.step_minibatches(dev(all_rows[t:t + 1], torch.int32))
        else:
            h.step_minibatches(dev(all_rows, torch.int32))
        assert h.last_path == (B.PATH_PERSISTENT if path == 0 else B.PATH_LAUNCHES)
        assert h.poll() == 0
        outs.append(h.get_state_host())
    for u, v in zip(*outs):
        np.testing.assert_array_equal(u, v)
    st = make_oracle_state(oracle32, w, k=k); st.init(0)
    for t in range(steps):
        st.step_minibatch(all_rows[t])
    assert rel_l2(outs[0][0], st.x) <= 1e-4


def test_full_batch_in_order_matches_the_deterministic_step(B, oracle32):
    # tau = m_i with the identity order visits the same rows in the same order as the full gradient: the same bits,
    # on the launch path (same tiles) and on the persistent path (same cluster shape, rows from global memory)
    w = inputs.config(0)
    m = int(np.min(np.diff(w.row_offsets)))
    batch = dev(np.tile(np.arange(m, dtype=np.int32), (w.n, 1)), torch.int32)
    for path in (B.PATH_LAUNCHES, B.PATH_PERSISTENT):
        a = make_gpu(w, k=1, path=path); b = make_gpu(w, k=1, path=path)
        if path == B.PATH_PERSISTENT:
            for h in (a, b):
                h.set_persistent_shape(2, 8, 2); h.set_persistent_threads(256)
        a.init(0); b.init(0)
        for _ in range(10):
            a.step(1); b.step_minibatch(batch)
        assert a.last_path == path and b.last_path == path
        for u, v in zip(a.get_state_host(), b.get_state_host()):
            np.testing.assert_array_equal(u, v)


def test_changing_tau_rebuilds_the_tile_table(B, oracle32):
    w = inputs.config(0)
    h = make_gpu(w, k=w.d); st = make_oracle_state(oracle32, w, k=w.d)
    h.init(1); st.init(1)
    for t, tau in enumerate((3, 40, 3, 17)):
        batch = inputs.minibatch_rows(2, t, w.row_offsets, tau)
        h.step_minibatch(dev(batch, torch.int32)); st.step_minibatch(batch)
        assert rel_l2(h.get_state_host()[0], st.x) <= 1e-5
        assert rel_l2(h.get_state_host()[1], st.g) <= 1e-4


@pytest.mark.parametrize("path", [1, 2], ids=["launches", "persistent"])
def test_bad_rows_are_reported_not_read(path, B):
    w = inputs.config(0)
    h = make_gpu(w, path=path)
    h.init(0)
    m = int(np.min(np.diff(w.row_offsets)))
    with pytest.raises(Exception):
        h.step_minibatch(dev(np.zeros((w.n, m + 1), dtype=np.int32), torch.int32))    # tau > m_i: refused on the host
    bad = np.zeros((w.n, 4), dtype=np.int32); bad[1, 2] = m; bad[2, 0] = -1         # outside the shard
    h.step_minibatch(dev(bad, torch.int32))
    torch.cuda.synchronize()
    assert h.poll() == 1          # EF21_ERR_INVALID_ARG
    h.clear_status()
    assert h.poll() == 0
