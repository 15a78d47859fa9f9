"""GPU parity for EF, the original error feedback method (Algorithm 4): iterates x^t and errors e_i^t
against the oracle, which runs the algorithm in the paper's own order."""
import os

import numpy as np
import pytest
import torch

import ef21_inputs as inputs
import oracle as oracle_mod
from gpu_util import dev, make_gpu, rel_l2

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def B():
    from paper_2106_05203_b200 import binding
    return binding


def _ef_oracle(o, w, k=None):
    return oracle_mod.EFState(o, w.n, w.d, k or w.k, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)


def test_hand_worked_run_on_gpu(B):
    from test_oracle_pins import _read_kv
    kv = _read_kv(os.path.join(GOLDEN, "alg4_hand_example.txt"))
    V = dev(np.array([kv["grad1"], kv["grad2"]], dtype=np.float32))
    h = B.EF21(2, 3, 1, kv["gamma"][0])
    h.set_variant(B.VARIANT_EF)
    h.init_grads(None, B.INIT_ZERO)
    for t in (1, 2, 3):
        h.step_grads(V, 1)
        x, _, e, li, lv = h.get_state_host()
        np.testing.assert_array_equal(x, kv[f"x{t}"])
        np.testing.assert_array_equal(e, [kv[f"e1_{t}"], kv[f"e2_{t}"]])
        np.testing.assert_array_equal(li[:, 0], kv[f"idx{t - 1}"])      # the messages that moved x^{t-1} to x^t
        np.testing.assert_array_equal(lv[:, 0], kv[f"val{t - 1}"])
    assert h.poll() == 0


@pytest.mark.parametrize("n,d,k", [(5, 300, 7), (3, 5000, 40), (20, 123, 16), (4, 300000, 300)])
def test_supplied_gradients_bit_exact(n, d, k, B, oracle32):
    # a changing gradient sequence, with ties (quantised entries) and coordinates hit by several workers
    rng = np.random.default_rng(d + k)
    gamma = 0.05
    T = 6
    Vs = [(np.round(rng.standard_normal((n, d)) * 8) / 8).astype(np.float32) for _ in range(T + 1)]
    h = B.EF21(n, d, k, gamma); h.set_variant(B.VARIANT_EF)
    h.init_grads(None, B.INIT_ZERO)
    st = oracle_mod.EFState(oracle32, n, d, k, gamma)
    st.init_from_grads(Vs[0])
    for t in range(T):
        sent_idx, sent_val = st.idx.copy(), st.val.copy()          # w^t
        h.step_grads(dev(Vs[t]), 1)                                # uses grad f_i(x^t)
        st.step_grads(Vs[t + 1], 1)                                # ends with the gradients at x^{t+1}
        x, _, e, li, lv = h.get_state_host()
        np.testing.assert_array_equal(li, sent_idx, err_msg=f"step {t}: message indices")
        np.testing.assert_array_equal(lv.view(np.uint32), sent_val.view(np.uint32), err_msg=f"step {t}: message values")
        np.testing.assert_array_equal(e.view(np.uint32), st.e.view(np.uint32), err_msg=f"step {t}: e_i")
        np.testing.assert_array_equal(x.view(np.uint32), st.x.view(np.uint32), err_msg=f"step {t}: x")
    assert h.poll() == 0


def test_supplied_gradients_multi_step_call_equals_single_steps(B):
    rng = np.random.default_rng(3)
    n, d, k = 6, 2000, 25
    V = dev(rng.standard_normal((n, d)).astype(np.float32))
    outs = []
    for chunks in ((5,), (1, 1, 1, 1, 1)):
        h = B.EF21(n, d, k, 0.1); h.set_variant(B.VARIANT_EF)
        h.init_grads(None, B.INIT_ZERO)
        for s in chunks:
            h.step_grads(V, s)
        x, _, e, _, _ = h.get_state_host()
        outs.append((x, e))
    np.testing.assert_array_equal(outs[0][0].view(np.uint32), outs[1][0].view(np.uint32))
    np.testing.assert_array_equal(outs[0][1].view(np.uint32), outs[1][1].view(np.uint32))


@pytest.mark.parametrize("path", [1, 2])
@pytest.mark.parametrize("cfg,k", [(0, 4), (1, 1), (2, 16)])
def test_logistic_ef_tracks_the_oracle(cfg, k, path, B, oracle32, oracle64):
    # launch-per-stage kernels (path 1) and the persistent cluster kernel (path 2)
    w = inputs.config(cfg, k=k)
    h = make_gpu(w, k=k, path=path); h.set_variant(B.VARIANT_EF)
    h.init(B.INIT_ZERO)
    st = _ef_oracle(oracle32, w, k=k)
    st.init()
    rebased = 0
    for t in range(40):
        x_old, e_old = st.x.copy(), st.e.copy()
        sent_idx = st.idx.copy()
        h.step(1); st.step(1)
        x, _, e, li, _ = h.get_state_host()
        if not np.array_equal(li, sent_idx):
            # only a near-tie of the compressed vector may change a pick; then continue from the oracle's state
            p = e_old.astype(np.float64) + w.gamma * oracle64.all_grads(w.A, w.y, w.row_offsets, x_old, w.lam)
            for i in range(w.n):
                kth = np.sort(np.abs(p[i]))[::-1][w.k - 1]
                for j in set(li[i].tolist()) ^ set(sent_idx[i].tolist()):
                    assert abs(abs(p[i][j]) - kth) <= 4e-5 * np.max(np.abs(p[i])), (t, i, j)
            rebased += 1
            h.set_state(dev(st.x), None, dev(st.e))
            continue
        assert rel_l2(x, st.x) <= 1e-4
        assert np.max(np.abs(e - st.e)) <= 1e-5 * max(np.max(np.abs(st.e)), w.gamma * 1.0)
        h.set_state(dev(st.x), None, dev(st.e))
    assert rebased <= 4
    assert h.last_path == path and h.poll() == 0


@pytest.mark.parametrize("path", [1, 2])
def test_free_running_ef_paper_shape(path, B, oracle32):
    w = inputs.config(1)
    h = make_gpu(w, path=path); h.set_variant(B.VARIANT_EF)
    h.init(B.INIT_ZERO)
    st = _ef_oracle(oracle32, w)
    st.init()
    h.step(60); st.step(60)
    assert h.last_path == path
    x = h.get_state_host()[0]
    assert rel_l2(x, st.x) <= 1e-4
    assert h.eval()[0] == pytest.approx(st.loss(), rel=1e-4)


def test_persistent_ef_many_steps_in_one_launch_equal_single_steps(B):
    w = inputs.config(2, k=4)
    outs = []
    for chunks in ((12,), (1,) * 12):
        h = make_gpu(w, k=4, path=2); h.set_variant(B.VARIANT_EF)
        h.init(B.INIT_ZERO)
        for s_ in chunks:
            h.step(s_)
        assert h.last_path == 2
        outs.append(h.get_state_host())
    for a_, b_ in zip(outs[0], outs[1]):
        np.testing.assert_array_equal(a_, b_)


def test_ef_has_no_minibatch_step(B):
    w = inputs.config(0)
    h = make_gpu(w); h.set_variant(B.VARIANT_EF)
    h.init(B.INIT_ZERO)
    batch = dev(inputs.minibatch_rows(0, 0, w.row_offsets, 8), dtype=torch.int32)
    with pytest.raises(B.Ef21Error) as e:
        h.step_minibatch(batch)
    assert e.value.status == 7
