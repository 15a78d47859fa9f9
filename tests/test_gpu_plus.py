"""GPU parity for EF21+ (Algorithm 3): the choice between the plain and the Markov compressor, the
resulting worker states and the recomputed average, against the oracle."""
import os

import numpy as np
import pytest

import ef21_inputs as inputs
import oracle as oracle_mod
from gpu_util import dev, make_gpu, make_oracle_state, rel_l2, set_gpu_state_from_oracle

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def B():
    from paper_2106_05203_b200 import binding
    return binding


def _assert_bitwise(h, st, what):
    x, g, gi, li, lv = h.get_state_host()
    np.testing.assert_array_equal(h.get_plus_choice(), st.choice, err_msg=f"{what}: choice")
    np.testing.assert_array_equal(li, st.idx, err_msg=f"{what}: idx")
    np.testing.assert_array_equal(lv.view(np.uint32), st.val.view(np.uint32), err_msg=f"{what}: val")
    np.testing.assert_array_equal(gi.view(np.uint32), st.gi.view(np.uint32), err_msg=f"{what}: g_i")
    np.testing.assert_array_equal(g.view(np.uint32), st.g.view(np.uint32), err_msg=f"{what}: g")
    np.testing.assert_array_equal(x.view(np.uint32), st.x.view(np.uint32), err_msg=f"{what}: x")


def test_hand_worked_round_on_gpu(B):
    from test_oracle_pins import _read_kv
    kv = _read_kv(os.path.join(GOLDEN, "alg3_hand_example.txt"))
    h = B.EF21(2, 2, 1, 0.5)
    h.set_variant(B.VARIANT_EF21_PLUS)
    h.set_state(dev(np.zeros(2, np.float32)), dev(np.zeros(2, np.float32)),
                dev(np.array([kv["g1"], kv["g2"]], dtype=np.float32)))
    h.step_grads(dev(np.array([kv["grad1"], kv["grad2"]], dtype=np.float32)), 1)
    x, g, gi, li, lv = h.get_state_host()
    np.testing.assert_array_equal(gi, [kv["new_g1"], kv["new_g2"]])
    np.testing.assert_array_equal(g, kv["new_g"])
    np.testing.assert_array_equal(h.get_plus_choice(), kv["choice"])
    np.testing.assert_array_equal(li[:, 0], kv["idx"])
    np.testing.assert_array_equal(lv[:, 0], kv["val"])


@pytest.mark.parametrize("n,d,k", [(5, 300, 7), (3, 5000, 40), (4, 300000, 300)])
def test_supplied_gradients_both_branches_bit_exact(n, d, k, B, oracle32):
    # a changing gradient sequence with jumps: some rounds keep the Markov compressor, others restart from C(grad)
    rng = np.random.default_rng(d)
    h = B.EF21(n, d, k, 0.05); h.set_variant(B.VARIANT_EF21_PLUS)
    st = oracle_mod.State(oracle32, n, d, k, 0.05)
    h.init_grads(None, 1); st.init(1)
    base = rng.standard_normal((n, d)).astype(np.float32)
    seen = set()
    for t in range(8):
        scale = np.float32(1.0 if t % 3 else 25.0)
        V = (base * scale + 0.01 * rng.standard_normal((n, d))).astype(np.float32)
        h.step_grads(dev(V), 1); st.plus_step_grads(V, 1)
        _assert_bitwise(h, st, f"step {t}")
        seen |= set(st.choice.tolist())
    assert seen == {0, 1}
    assert h.poll() == 0


@pytest.mark.parametrize("path", [1, 2])
@pytest.mark.parametrize("cfg,k", [(0, 4), (1, 1), (2, 16)])
def test_logistic_ef21_plus_tracks_the_oracle(cfg, k, path, B, oracle32):
    # launch-per-stage kernels (path 1) and the persistent cluster kernel (path 2)
    w = inputs.config(cfg, k=k)
    h = make_gpu(w, k=k, path=path); h.set_variant(B.VARIANT_EF21_PLUS)
    st = make_oracle_state(oracle32, w, k=k)
    h.init(0); st.init(0)
    rebased = 0
    for t in range(30):
        gi_old = st.gi.copy()
        h.step(1); st.plus_step(1)
        assert h.last_path == path
        x, g, gi, li, lv = h.get_state_host()
        if not (np.array_equal(h.get_plus_choice(), st.choice) and np.array_equal(li, st.idx)):
            # only a near-tie (between two entries, or between the two distortions) may change a decision
            grads = st.grads().astype(np.float64)
            for i in range(w.n):
                if h.get_plus_choice()[i] != st.choice[i]:
                    # the two distortions of Algorithm 3 must then be within the effect of the gradient tolerance
                    # of each other: M_i = ||g_i + C(grad_i - g_i) - grad_i||^2, B_i = ||C(grad_i) - grad_i||^2
                    vm = grads[i] - gi_old[i]
                    im, _ = oracle32.topk(vm.astype(np.float32), k)
                    ib, _ = oracle32.topk(grads[i].astype(np.float32), k)
                    rest_m = vm.copy(); rest_m[im] = 0.0
                    rest_b = grads[i].copy(); rest_b[ib] = 0.0
                    M, Bd = float(rest_m @ rest_m), float(rest_b @ rest_b)
                    assert abs(M - Bd) <= 1e-4 * max(M, Bd), (t, i, M, Bd)
                    continue
                v = grads[i] - gi_old[i] if st.choice[i] == 0 else grads[i]
                kth = np.sort(np.abs(v))[::-1][k - 1]
                for j in set(li[i].tolist()) ^ set(st.idx[i].tolist()):
                    assert abs(abs(v[j]) - kth) <= 2e-5 * (np.max(np.abs(grads[i])) + 1e-30), (t, i, j)
            rebased += 1
        else:
            assert rel_l2(x, st.x) <= 1e-4 or np.linalg.norm(st.x) == 0
            assert np.max(np.abs(gi - st.gi)) <= 1e-5 * np.max(np.abs(st.gi))
            assert np.max(np.abs(g - st.g)) <= 1e-5 * np.max(np.abs(st.gi))      # g is a mean of the g_i: their scale
        set_gpu_state_from_oracle(h, st)
    assert rebased <= 3
    assert h.poll() == 0


@pytest.mark.parametrize("path", [1, 2])
def test_free_running_ef21_plus_paper_shape(path, B, oracle32):
    w = inputs.config(1)
    h = make_gpu(w, path=path); h.set_variant(B.VARIANT_EF21_PLUS)
    st = make_oracle_state(oracle32, w)
    h.init(0); st.init(0)
    h.step(60); st.plus_step(60)
    assert h.last_path == path
    x = h.get_state_host()[0]
    assert rel_l2(x, st.x) <= 1e-4
    assert h.eval()[0] == pytest.approx(st.loss(), rel=1e-4)


def test_persistent_ef21_plus_many_steps_in_one_launch_equal_single_steps(B):
    w = inputs.config(2, k=4)
    outs = []
    for chunks in ((12,), (1,) * 12):
        h = make_gpu(w, k=4, path=2); h.set_variant(B.VARIANT_EF21_PLUS)
        h.init(0)
        for s_ in chunks:
            h.step(s_)
        outs.append(h.get_state_host() + (h.get_plus_choice(),))
    for a_, b_ in zip(outs[0], outs[1]):
        np.testing.assert_array_equal(a_, b_)


@pytest.mark.parametrize("n,d,k", [(6, 64, 3), (20, 112, 1), (40, 100, 2)], ids=["n6", "n20", "n40"])
def test_persistent_ef21_plus_takes_the_plain_branch(n, d, k, B, oracle32):
    """Workers whose g_i is far from their gradient must fall back to the plain compressor (B_i < M_i, Algorithm 3):
    their row of the replicas restarts from zero.  Every other worker is put there by hand, the rest keep their state,
    so one launch sees both branches side by side (n = 40: more workers than one ballot covers)."""
    w = inputs.make_logistic("plusbranch", n=n, d=d, N=n * 30, k=k, seed=4000 + n, features="gauss", flip=0.1, gamma=0.05, T=10)
    h = make_gpu(w, k=k, path=2); h.set_variant(B.VARIANT_EF21_PLUS)
    st = make_oracle_state(oracle32, w, k=k)
    h.init(0); st.init(0)
    rng = np.random.default_rng(n)
    seen = set()
    for t in range(6):
        if t % 2 == 0:
            st.gi[t // 2 % 2::2] = (25.0 * rng.standard_normal(st.gi[t // 2 % 2::2].shape)).astype(np.float32)
        set_gpu_state_from_oracle(h, st)
        gi_old = st.gi.copy()
        h.step(1); st.plus_step(1)
        assert h.last_path == B.PATH_PERSISTENT
        x, g, gi, li, lv = h.get_state_host()
        choice = h.get_plus_choice()
        for i in np.flatnonzero(choice != st.choice):
            # only two distortions within the effect of the gradient tolerance of each other may be ordered differently
            gd = st.grads()[i].astype(np.float64)
            vm = gd - gi_old[i]
            im, _ = oracle32.topk(vm.astype(np.float32), k)
            ib, _ = oracle32.topk(gd.astype(np.float32), k)
            rest_m = vm.copy(); rest_m[im] = 0.0
            rest_b = gd.copy(); rest_b[ib] = 0.0
            M, Bd = float(rest_m @ rest_m), float(rest_b @ rest_b)
            assert abs(M - Bd) <= 1e-4 * max(M, Bd), (t, i, M, Bd)
        if not np.array_equal(choice, st.choice):
            continue
        if t % 2 == 0:
            assert np.all(st.choice[t // 2 % 2::2] == 1), "a g_i of norm 25 sqrt(d) must lose against the plain compressor"
        seen |= set(st.choice.tolist())
        grads = st.grads()
        for i in range(n):
            tol = 1e-5 * np.max(np.abs(grads[i]))
            if st.choice[i] == 1:
                # C(grad_i): index set up to near-ties, values within the gradient tolerance, all other entries exactly 0
                assert np.count_nonzero(gi[i]) <= k
                if np.array_equal(li[i], st.idx[i]):
                    assert np.max(np.abs(lv[i] - st.val[i])) <= tol
                    assert np.max(np.abs(gi[i] - st.gi[i])) <= tol
            elif np.array_equal(li[i], st.idx[i]):
                assert np.max(np.abs(gi[i] - st.gi[i])) <= tol + 4e-6 * np.max(np.abs(gi_old[i]))
        assert np.max(np.abs(g - st.g)) <= 1e-5 * max(np.max(np.abs(st.gi)), 1e-30)
        assert rel_l2(x, st.x) <= 1e-5
    assert seen == {0, 1}
    assert h.poll() == 0
