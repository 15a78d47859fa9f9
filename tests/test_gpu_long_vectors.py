"""GPU parity for long vectors (the one-pass Top-k path, d >= 2^18): bit-exact against the oracle,
including the inputs that defeat the sampled threshold and must fall back to the exact
whole-vector selection, and the full-size supplied-gradient workload (n = 64, d = 4,194,304,
k = 4,194) on sampled workers."""
import numpy as np
import pytest
import torch

import ef21_inputs as inputs
import oracle as oracle_mod
from gpu_util import assert_state_bitwise, dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2106_05203_b200 import binding
    return binding


def _long_cases():
    rng = np.random.default_rng(77)
    cases = []
    cases.append(("student-262144-k1", inputs.stress_vector(5, 0, 262144), 1))
    cases.append(("student-262144-k262", inputs.stress_vector(5, 1, 262144), 262))
    cases.append(("student-1m-k6144", inputs.stress_vector(5, 2, 1 << 20), 6144))
    cases.append(("student-1m-k8192-multipass", inputs.stress_vector(5, 2, 1 << 20), 8192))
    cases.append(("gauss-unaligned-300001", rng.standard_normal(300001).astype(np.float32), 100))
    cases.append(("gauss-ragged-region-266245", rng.standard_normal(266245).astype(np.float32), 3000))
    v = (rng.integers(-4, 5, 400000)).astype(np.float32) * np.float32(0.25)        # nine magnitudes: huge tie classes
    cases.append(("quantised-fallback", v, 5000))
    v = np.zeros(300000, dtype=np.float32); v[rng.choice(300000, 100, replace=False)] = rng.standard_normal(100)
    cases.append(("sparse-fewer-nonzeros-than-k", v, 300))
    v = (rng.standard_normal(500000) * 1e-3).astype(np.float32)
    v[7 * 4096:8 * 4096] = rng.standard_normal(4096).astype(np.float32) * 10        # all large entries in one region
    cases.append(("clustered-region-overflow", v, 3000))
    cases.append(("all-equal", np.full(270000, -1.5, dtype=np.float32), 4000))
    return cases


@pytest.mark.parametrize("name,v,k", _long_cases(), ids=[c[0] for c in _long_cases()])
def test_long_topk_bit_exact(name, v, k, B, oracle32):
    idx, val = B.topk(dev(v), k)
    oi, ov = oracle32.topk(v, k)
    np.testing.assert_array_equal(idx.cpu().numpy()[0], oi)
    np.testing.assert_array_equal(val.cpu().numpy()[0].view(np.uint32), ov.view(np.uint32))


def test_long_topk_batch(B, oracle32):
    V = np.stack([inputs.stress_vector(9, i, 400000) for i in range(6)])
    idx, val = B.topk(dev(V), 400)
    for i in range(6):
        oi, ov = oracle32.topk(V[i], 400)
        np.testing.assert_array_equal(idx[i].cpu().numpy(), oi)
        np.testing.assert_array_equal(val[i].cpu().numpy(), ov)


@pytest.mark.parametrize("n,d,k,mode", [(8, 300000, 300, 1), (64, 262144, 262, 1), (3, 524289, 2000, 0)])
def test_supplied_gradients_long_bit_exact(n, d, k, mode, B, oracle32):
    V = np.stack([inputs.stress_vector(200 + n, i, d) for i in range(n)])
    h = B.EF21(n, d, k, 0.01)
    st = oracle_mod.State(oracle32, n, d, k, 0.01)
    Vd = dev(V)
    h.init_grads(Vd, mode); st.init_from_grads(V, mode)
    assert_state_bitwise(h, st, "init")
    for t in range(4):
        h.step_grads(Vd, 1); st.step_grads(V, 1)
        assert_state_bitwise(h, st, f"step {t}")
    assert h.fallback_count() == 0, "the sampled threshold should never miss on this input"
    # the multi-pass radix select gives the same bits
    h2 = B.EF21(n, d, k, 0.01); h2.set_topk_algorithm(1)
    h2.init_grads(Vd, mode); h2.step_grads(Vd, 4)
    for a, b in zip(h.get_state_host(), h2.get_state_host()):
        np.testing.assert_array_equal(a, b)
    assert h.poll() == 0


def test_supplied_gradients_fallback_is_exact(B, oracle32):
    # vectors whose difference is heavily tied: every round goes through the whole-vector fallback
    n, d, k = 3, 270000, 500
    rng = np.random.default_rng(1)
    V = (rng.integers(-2, 3, (n, d))).astype(np.float32)
    h = B.EF21(n, d, k, 0.01); st = oracle_mod.State(oracle32, n, d, k, 0.01)
    h.init_grads(None, 1); st.init(1)
    h.step_grads(dev(V), 3); st.step_grads(V, 3)
    assert_state_bitwise(h, st, "tied input")
    assert h.fallback_count() > 0


def test_stress_workload_full_size_sampled_workers(B, oracle32):
    """n = 64, d = 4,194,304, k = 4,194 with the static Student-t vectors: the messages and g_i of
    sampled workers are compared bit for bit with the oracle run on that worker alone (workers
    only interact through g); g is checked against the mean of the g_i, x against the running sum
    of the g it was built from."""
    w = inputs.config(4)
    sampled = (0, 29, 63)
    V = torch.empty((w.n, w.d), dtype=torch.float32, device="cuda")
    host = {}
    for i in range(w.n):
        vi = w.worker_vector(i)
        if i in sampled:
            host[i] = vi
        V[i].copy_(torch.from_numpy(vi))
    h = B.EF21(w.n, w.d, w.k, w.gamma)
    h.init_grads(None, B.INIT_ZERO)
    solo = {i: oracle_mod.State(oracle32, 1, w.d, w.k, w.gamma) for i in sampled}
    x_expect = np.zeros(w.d, dtype=np.float64)
    g_prev = np.zeros(w.d, dtype=np.float32)
    for t in range(3):
        h.step_grads(V, 1)
        x, g, gi, li, lv = h.get_state()
        x_expect -= w.gamma * g_prev.astype(np.float64)
        for i in sampled:
            solo[i].step_grads(host[i][None, :], 1)
            np.testing.assert_array_equal(li[i].cpu().numpy(), solo[i].idx[0])
            np.testing.assert_array_equal(lv[i].cpu().numpy(), solo[i].val[0])
            np.testing.assert_array_equal(gi[i].cpu().numpy(), solo[i].gi[0])
        assert int((gi != 0).sum().item()) == w.n * w.k * (t + 1)           # k new coordinates per worker
        g_host = g.cpu().numpy()
        mean = gi.double().mean(dim=0).cpu().numpy()
        assert np.max(np.abs(g_host - mean)) <= 1e-6 * max(1.0, np.max(np.abs(mean)))
        assert np.max(np.abs(x.cpu().numpy() - x_expect)) <= 1e-6
        g_prev = g_host
    assert h.fallback_count() == 0
    assert h.poll() == 0
