"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each names the passage it
checks; together a dropped term, a wrong sign, a wrong index or a transposed
operand anywhere in the oracle fails at least one of them.
"""
import math
import os

import numpy as np
import pytest

import ef21_inputs as inputs
import oracle as oracle_mod

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------
# Objective and gradient (Section 5, Eq. 19)
# ---------------------------------------------------------------------------

def _read_closed_form_cases():
    cases = []
    with open(os.path.join(GOLDEN, "logistic_closed_form.txt")) as fh:
        for line in fh:
            if not line.startswith("case"):
                continue
            tok = line.split()
            fields, key = {}, None
            for t in tok[1:]:
                if t in ("A", "y", "x", "lam", "f", "grad"):
                    key = t
                    fields[key] = []
                else:
                    fields[key].append(float(t))
            cases.append(fields)
    return cases


@pytest.mark.parametrize("case", _read_closed_form_cases())
def test_loss_and_grad_closed_form(case, oracle64):
    A = np.array([case["A"]], dtype=np.float32)
    y = np.array(case["y"], dtype=np.float32)
    x = np.array(case["x"], dtype=np.float64)
    lam = case["lam"][0]
    assert oracle64.local_loss(A, y, x, lam) == pytest.approx(case["f"][0], rel=1e-14, abs=1e-15)
    np.testing.assert_allclose(oracle64.local_grad(A, y, x, lam), case["grad"], rtol=1e-14, atol=1e-15)


def test_grad_matches_central_differences(oracle64):
    w = inputs.config(0)
    rng = np.random.default_rng(123)
    x = rng.standard_normal(w.d) * 0.7
    for i in range(w.n):
        Ai = w.A[w.row_offsets[i]:w.row_offsets[i + 1]]
        yi = w.y[w.row_offsets[i]:w.row_offsets[i + 1]]
        g = oracle64.local_grad(Ai, yi, x, w.lam)
        h = 1e-6
        fd = np.empty(w.d)
        for j in range(w.d):
            e = np.zeros(w.d); e[j] = h
            fd[j] = (oracle64.local_loss(Ai, yi, x + e, w.lam) - oracle64.local_loss(Ai, yi, x - e, w.lam)) / (2 * h)
        assert np.max(np.abs(fd - g)) <= 1e-8 * max(1.0, np.max(np.abs(g)))


def test_loss_and_grad_at_zero(oracle64):
    # f(0) = log 2 for every shard; grad f_i(0) = -(1/(2 m_i)) A_i^T y_i (regulariser vanishes).
    w = inputs.config(1)
    x = np.zeros(w.d)
    assert oracle64.loss(w.A, w.y, w.row_offsets, x, w.lam) == pytest.approx(math.log(2.0), rel=1e-14)
    grads = oracle64.all_grads(w.A, w.y, w.row_offsets, x, w.lam)
    for i in (0, 7, w.n - 1):
        r0, r1 = w.row_offsets[i], w.row_offsets[i + 1]
        expect = -(w.A[r0:r1].astype(np.float64).T @ w.y[r0:r1].astype(np.float64)) / (2.0 * (r1 - r0))
        np.testing.assert_allclose(grads[i], expect, rtol=1e-13, atol=1e-15)


def test_loss_is_mean_of_local_losses_with_own_row_counts(oracle64):
    # Eq. 1: f = (1/n) sum f_i, f_i averaged over its own m_i; uneven shards expose a wrong normaliser.
    w = inputs.config(0)
    off = np.array([0, 10, 60, 61, 200], dtype=np.int64)
    x = np.linspace(-1, 1, w.d)
    parts = [oracle64.local_loss(w.A[off[i]:off[i + 1]], w.y[off[i]:off[i + 1]], x, w.lam) for i in range(4)]
    assert oracle64.loss(w.A, w.y, off, x, w.lam) == pytest.approx(np.mean(parts), rel=1e-14)
    z = w.A[10:60].astype(np.float64) @ x
    direct = np.mean(np.logaddexp(0.0, -w.y[10:60] * z)) + w.lam * np.sum(x * x / (1 + x * x))
    assert parts[1] == pytest.approx(direct, rel=1e-13)


def test_large_margins_do_not_overflow(oracle64):
    A = np.array([[1000.0], [1000.0]], dtype=np.float32)
    y = np.array([1.0, -1.0], dtype=np.float32)
    x = np.array([1.0])
    f = oracle64.local_loss(A, y, x, 0.0)
    g = oracle64.local_grad(A, y, x, 0.0)
    assert f == pytest.approx(500.0, rel=1e-12)       # (0 + 1000)/2
    assert g[0] == pytest.approx(500.0, rel=1e-12)    # (0 + 1000)/2


# ---------------------------------------------------------------------------
# Top-k (Section 2.1, Eq. 3)
# ---------------------------------------------------------------------------

def _brute_topk(v, k):
    mag = np.abs(v.astype(np.float64))
    order = np.lexsort((np.arange(v.size), -mag))      # |v| descending, index ascending
    keep = np.sort(order[:k])
    return keep.astype(np.int32), v[keep]


@pytest.mark.parametrize("d,k", [(1, 1), (7, 3), (64, 4), (1000, 1), (1000, 999), (4096, 517)])
def test_topk_matches_brute_force(d, k, oracle32):
    rng = np.random.default_rng(d * 31 + k)
    v = rng.standard_normal(d).astype(np.float32)
    v[rng.integers(0, d, size=max(1, d // 5))] = np.float32(0.5)   # plant exact ties
    idx, val = oracle32.topk(v, k)
    bi, bv = _brute_topk(v, k)
    np.testing.assert_array_equal(idx, bi)
    np.testing.assert_array_equal(val, bv)


def test_topk_matches_brute_force_4m(oracle32):
    v = inputs.stress_vector(4, 0, 1 << 22)
    k = (1 << 22) // 1000
    idx, val = oracle32.topk(v, k)
    bi, bv = _brute_topk(v, k)
    np.testing.assert_array_equal(idx, bi)
    np.testing.assert_array_equal(val, bv)


def test_topk_tie_rule_and_signed_zero(oracle32):
    idx, val = oracle32.topk(np.array([2, -2, 2, 1], dtype=np.float32), 2)
    np.testing.assert_array_equal(idx, [0, 1]); np.testing.assert_array_equal(val, [2, -2])
    idx, _ = oracle32.topk(np.full(9, -3.0, dtype=np.float32), 4)
    np.testing.assert_array_equal(idx, [0, 1, 2, 3])
    v = np.array([0.0, -0.0, 0.0, 5.0, -0.0], dtype=np.float32)
    idx, val = oracle32.topk(v, 3)                     # fewer non-zeros than k: zeros by lowest index
    np.testing.assert_array_equal(idx, [0, 1, 3])
    assert np.signbit(val[1]) and not np.signbit(val[0]) and val[2] == 5.0
    v = np.array([1e-45, -3e-45, 0.0, 1e-45], dtype=np.float32)   # subnormals order by magnitude
    idx, _ = oracle32.topk(v, 2)
    np.testing.assert_array_equal(idx, [0, 1])


def test_topk_identity_when_k_equals_d(oracle32):
    v = np.random.default_rng(5).standard_normal(257).astype(np.float32)
    idx, val = oracle32.topk(v, v.size)
    np.testing.assert_array_equal(idx, np.arange(v.size))
    np.testing.assert_array_equal(val, v)


@pytest.mark.parametrize("d,k", [(64, 4), (300, 1), (1000, 250)])
def test_topk_contraction_bound(d, k, oracle64):
    # Eq. 3 with alpha = k/d: ||C(v) - v||^2 <= (1 - k/d) ||v||^2, equality for constant magnitude.
    rng = np.random.default_rng(d + k)
    for v in (rng.standard_normal(d), rng.standard_t(3, d), np.where(rng.random(d) < 0.5, -1.5, 1.5)):
        idx, val = oracle64.topk(v, k)
        c = np.zeros(d); c[idx] = val
        lhs, rhs = np.sum((c - v) ** 2), (1 - k / d) * np.sum(v ** 2)
        assert lhs <= rhs * (1 + 1e-12)
    idx, val = oracle64.topk(np.where(np.arange(d) % 2 == 0, -1.5, 1.5), k)
    c = np.zeros(d); c[idx] = val
    v = np.where(np.arange(d) % 2 == 0, -1.5, 1.5)
    assert np.sum((c - v) ** 2) == pytest.approx((1 - k / d) * np.sum(v ** 2), rel=1e-12)


# ---------------------------------------------------------------------------
# Algorithm 2 (the loop), Algorithm 1, Section 3.1
# ---------------------------------------------------------------------------

def _read_hand_example():
    scal, vec = {}, {}
    with open(os.path.join(GOLDEN, "alg2_hand_example.txt")) as fh:
        for line in fh:
            tok = line.split()
            if not tok or tok[0].startswith("#"):
                continue
            if tok[0] in ("n", "d", "k", "gamma"):
                scal[tok[0]] = float(tok[1])
            elif tok[0] in ("V1", "V2"):
                vec[tok[0]] = [float(t) for t in tok[1:]]
            else:
                vec[(tok[0], tok[1])] = [float(t) for t in tok[2:]]
    return scal, vec


@pytest.mark.parametrize("precision", ["f32", "f64"])
def test_alg2_hand_worked_example(precision):
    o = oracle_mod.Oracle(precision)
    scal, vec = _read_hand_example()
    n, d, k = int(scal["n"]), int(scal["d"]), int(scal["k"])
    V = np.array([vec["V1"], vec["V2"]])
    st = oracle_mod.State(o, n, d, k, scal["gamma"])
    st.init_from_grads(V, mode=0)
    for t in range(4):
        tag = f"t{t}"
        np.testing.assert_array_equal(st.x, vec[(tag, "x")])
        np.testing.assert_array_equal(st.gi[0], vec[(tag, "g1")])
        np.testing.assert_array_equal(st.gi[1], vec[(tag, "g2")])
        np.testing.assert_array_equal(st.g, vec[(tag, "g")])
        if t > 0:
            np.testing.assert_array_equal(st.idx[:, 0], vec[(tag, "idx")])
            np.testing.assert_array_equal(st.val[:, 0], vec[(tag, "val")])
        st.step_grads(V, 1)


def test_k_equals_d_is_gradient_descent(oracle64):
    # Section 5.2: "GD ... can be thought of as EF21 with k = d".
    w = inputs.config(0)
    st = oracle_mod.State(oracle64, w.n, w.d, w.d, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(0)
    x = w.x0.astype(np.float64)
    for _ in range(30):
        grad = oracle64.all_grads(w.A, w.y, w.row_offsets, x, w.lam).mean(axis=0)
        np.testing.assert_allclose(st.g, grad, rtol=0, atol=1e-14)
        x = x - w.gamma * grad
        st.step(1)
        np.testing.assert_allclose(st.x, x, rtol=0, atol=1e-13)
        np.testing.assert_allclose(st.gi, oracle64.all_grads(w.A, w.y, w.row_offsets, st.x, w.lam),
                                   rtol=0, atol=1e-14)


def test_k_equals_d_fp32_state_tracks_gradient(oracle32):
    # In fp32, g + (a - g) differs from a by a couple of ulps at most; init (Top-d of the gradient) is exact.
    w = inputs.config(0)
    st = oracle_mod.State(oracle32, w.n, w.d, w.d, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(0)
    np.testing.assert_array_equal(st.gi, oracle32.all_grads(w.A, w.y, w.row_offsets, st.x, w.lam))
    for _ in range(10):
        st.step(1)
        grads = oracle32.all_grads(w.A, w.y, w.row_offsets, st.x, w.lam)
        assert np.max(np.abs(st.gi - grads)) <= 4 * np.finfo(np.float32).eps * np.max(np.abs(grads))


def test_single_node_is_algorithm_1(oracle64):
    # Algorithm 1: x^{t+1} = x^t - gamma g^t;  g^{t+1} = g^t + C(grad f(x^{t+1}) - g^t);  g^0 = C(grad f(x^0)).
    w = inputs.config(0)
    off = np.array([0, w.N], dtype=np.int64)
    k = 3
    st = oracle_mod.State(oracle64, 1, w.d, k, w.gamma, w.lam, w.A, w.y, off, w.x0)
    st.init(0)

    def C(v):
        keep, vals = _brute_topk(v, k)
        c = np.zeros_like(v); c[keep] = vals
        return c

    x = w.x0.astype(np.float64)
    g = C(oracle64.local_grad(w.A, w.y, x, w.lam))
    for _ in range(25):
        np.testing.assert_allclose(st.g, g, rtol=0, atol=1e-15)
        np.testing.assert_allclose(st.gi[0], g, rtol=0, atol=1e-15)
        x = x - w.gamma * g
        g = g + C(oracle64.local_grad(w.A, w.y, x, w.lam) - g)
        st.step(1)
        np.testing.assert_allclose(st.x, x, rtol=0, atol=1e-14)


@pytest.mark.parametrize("mode", [0, 1, 2])
def test_master_average_and_one_step_distortion(mode, oracle64):
    # Algorithm 2, last loop line: g^t = (1/n) sum_i g_i^t at every t.
    # Proof of Lemma 2, third line: ||g_i^{t+1} - grad f_i(x^{t+1})||^2 <= (1 - k/d) ||grad f_i(x^{t+1}) - g_i^t||^2.
    w = inputs.config(0)
    st = oracle_mod.State(oracle64, w.n, w.d, w.k, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(mode)
    if mode == 1:
        assert not st.gi.any() and not st.g.any()
    if mode == 2:
        np.testing.assert_allclose(st.gi, st.grads(), atol=1e-16)
    for _ in range(40):
        gi_old = st.gi.copy()
        st.step(1)
        np.testing.assert_allclose(st.g, st.gi.mean(axis=0), rtol=0, atol=1e-14)
        grads = st.grads()
        lhs = np.sum((st.gi - grads) ** 2, axis=1)
        rhs = (1 - w.k / w.d) * np.sum((grads - gi_old) ** 2, axis=1)
        assert np.all(lhs <= rhs * (1 + 1e-12) + 1e-30)
        # the message is exactly the compressed difference, and exactly k coordinates moved
        for i in range(w.n):
            bi, bv = _brute_topk(grads[i] - gi_old[i], w.k)
            np.testing.assert_array_equal(st.idx[i], bi)
            np.testing.assert_allclose(st.val[i], bv, rtol=0, atol=0)
            changed = np.flatnonzero(st.gi[i] != gi_old[i])
            assert set(changed) <= set(bi)


def test_theorem_1_lyapunov_descent_and_rate(oracle64):
    # With gamma at the bound of Theorem 1 (Eq. 13) the proof's Lyapunov function
    # f(x^t) - f_inf + (gamma/(2 theta)) G^t decreases by at least (gamma/2)||grad f(x^t)||^2 per step,
    # and the averaged squared gradient norm obeys Eq. 14 with f_inf >= 0.
    w = inputs.config(0)
    k = 4
    gamma = inputs.theory_gamma(w.A, w.row_offsets, w.lam, k)
    alpha = k / w.d
    theta = 1 - math.sqrt(1 - alpha)
    st = oracle_mod.State(oracle64, w.n, w.d, k, gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(0)
    T = 60
    f0 = st.loss()
    _, G0 = oracle64.diagnostics(w.A, w.y, w.row_offsets, st.x, w.lam, st.gi)
    f_prev, G_prev = f0, G0
    sq_norms = []
    for _ in range(T):
        nrm2, _ = oracle64.diagnostics(w.A, w.y, w.row_offsets, st.x, w.lam, st.gi)
        sq_norms.append(nrm2)
        st.step(1)
        f_new = st.loss()
        _, G_new = oracle64.diagnostics(w.A, w.y, w.row_offsets, st.x, w.lam, st.gi)
        lhs = f_new + gamma / (2 * theta) * G_new
        rhs = f_prev + gamma / (2 * theta) * G_prev - gamma / 2 * nrm2
        assert lhs <= rhs + 1e-13
        f_prev, G_prev = f_new, G_new
    assert np.mean(sq_norms) <= 2 * (f0 - 0.0) / (gamma * T) + G0 / (theta * T)


def test_diagnostics_closed_forms_at_the_origin(oracle64):
    # Section 3.3: G^t = (1/n) sum_i ||g_i^t - grad f_i(x^t)||^2.  At x = 0 the gradient of Eq. 19 is
    # grad f_i(0) = -A_i^T y_i / (2 m_i) (sigmoid(0) = 1/2, the regulariser's derivative vanishes), so with
    # g_i = 0:  G = (1/n) sum_i ||A_i^T y_i||^2 / (4 m_i^2)  and  ||grad f(0)||^2 = ||(1/n) sum_i A_i^T y_i / (2 m_i)||^2.
    # The two differ by where 1/n sits, so a dropped or misplaced 1/n in either fails here.
    w = inputs.config(0)
    off = w.row_offsets
    per_worker = []
    for i in range(w.n):
        Ai = w.A[off[i]:off[i + 1]].astype(np.float64)
        yi = w.y[off[i]:off[i + 1]].astype(np.float64)
        per_worker.append(-(Ai.T @ yi) / (2.0 * (off[i + 1] - off[i])))
    per_worker = np.array(per_worker)
    G_expect = np.sum(per_worker ** 2) / w.n
    nrm_expect = np.sum(np.mean(per_worker, axis=0) ** 2)
    zeros = np.zeros((w.n, w.d))
    nrm2, G = oracle64.diagnostics(w.A, w.y, off, np.zeros(w.d), w.lam, zeros)
    assert G == pytest.approx(G_expect, rel=1e-13)
    assert nrm2 == pytest.approx(nrm_expect, rel=1e-13)
    assert G > 2 * nrm2           # heterogeneous shards: the mean of squares is not the square of the mean


def test_diagnostics_zero_and_planted_distortion(oracle64):
    # G = 0 exactly when every g_i is the local gradient (initialisation g_i^0 = grad f_i(x^0), Section 3.3, last
    # paragraph); with g_i = grad f_i(x) + E_i for a planted E it is ||E||_F^2 / n whatever x is.
    w = inputs.config(0)
    rng = np.random.default_rng(5)
    x = rng.standard_normal(w.d) * 0.3
    grads = oracle64.all_grads(w.A, w.y, w.row_offsets, x, w.lam)
    nrm2, G = oracle64.diagnostics(w.A, w.y, w.row_offsets, x, w.lam, grads)
    assert G == 0.0
    assert nrm2 == pytest.approx(np.sum(np.mean(grads, axis=0) ** 2), rel=1e-13)
    E = np.zeros((w.n, w.d)); E[0, 3] = 0.5; E[2, 10] = -2.0; E[3, 63] = 1.0      # exactly representable
    _, G = oracle64.diagnostics(w.A, w.y, w.row_offsets, x, w.lam, grads + E)
    assert G == pytest.approx((0.25 + 4.0 + 1.0) / w.n, rel=1e-12)
    # a state built by the oracle in mode 2 (g_i^0 = grad f_i(x^0)) starts with G^0 = 0
    st = oracle_mod.State(oracle64, w.n, w.d, w.k, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(2)
    assert oracle64.diagnostics(w.A, w.y, w.row_offsets, st.x, w.lam, st.gi)[1] == 0.0


# ---------------------------------------------------------------------------
# Scaled Rand-k (Appendix: Lemma 8, Example 2)
# ---------------------------------------------------------------------------

def test_randk_exact_moments_over_all_subsets(oracle64):
    # Rand-k is in U(omega) with omega = d/k - 1: averaged over all C(d, k) equally likely sets, E C'(v) = v and
    # E||C'(v)||^2 = (d/k)||v||^2 = (1 + omega)||v||^2.  Its scaled version (Lemma 8, factor 1/(1 + omega) = k/d) keeps
    # the sampled entries as they are, has mean (k/d) v, and meets the bound of Eq. 3 with alpha = k/d with equality:
    # E||C(v) - v||^2 = (1 - k/d)||v||^2.
    import itertools
    rng = np.random.default_rng(2)
    for d, k in ((5, 2), (6, 3), (7, 1), (4, 4)):
        v = rng.standard_normal(d)
        sets = list(itertools.combinations(range(d), k))
        mean_unb = np.zeros(d); mean_sc = np.zeros(d); sq_unb = 0.0; dist_sc = 0.0
        for S in sets:
            iu, vu = oracle64.randk(v, S, unbiased=True)
            i_s, vs = oracle64.randk(v, S)
            np.testing.assert_array_equal(iu, S); np.testing.assert_array_equal(i_s, S)
            cu = np.zeros(d); cu[iu] = vu
            cs = np.zeros(d); cs[i_s] = vs
            mean_unb += cu; mean_sc += cs
            sq_unb += cu @ cu; dist_sc += (cs - v) @ (cs - v)
            np.testing.assert_array_equal(vs, v[list(S)])             # the two scalings cancel: the entries themselves
        m = len(sets)
        np.testing.assert_allclose(mean_unb / m, v, rtol=1e-13)
        np.testing.assert_allclose(mean_sc / m, (k / d) * v, rtol=1e-13)
        assert sq_unb / m == pytest.approx((d / k) * (v @ v), rel=1e-13)
        assert dist_sc / m == pytest.approx((1 - k / d) * (v @ v), rel=1e-13, abs=1e-15)


def test_randk_loop_k_equals_d_is_gradient_descent_and_mean_invariant(oracle64):
    # with S = all coordinates the scaled Rand-k is the identity, so Algorithm 2 is gradient descent (Section 5.2's
    # remark on k = d); with k < d the master's g stays the mean of the g_i and only the named coordinates move
    w = inputs.config(0)
    full = np.tile(np.arange(w.d, dtype=np.int32), (6, w.n, 1))
    st = oracle_mod.State(oracle64, w.n, w.d, w.d, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(2)
    x = np.array(w.x0, dtype=np.float64)
    g = oracle64.all_grads(w.A, w.y, w.row_offsets, x, w.lam).mean(axis=0)
    for t in range(6):
        x = x - w.gamma * g
        g = oracle64.all_grads(w.A, w.y, w.row_offsets, x, w.lam).mean(axis=0)
    st.step_randk(full)
    np.testing.assert_allclose(st.x, x, rtol=1e-12, atol=1e-14)
    k = 5
    sets = inputs.randk_sets(3, 12, w.n, w.d, k)
    st = oracle_mod.State(oracle64, w.n, w.d, k, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(1)
    for t in range(12):
        gi_old = st.gi.copy()
        st.step_randk(sets[t:t + 1])
        np.testing.assert_allclose(st.g, st.gi.mean(axis=0), rtol=1e-12, atol=1e-15)
        grads = st.grads()
        for i in range(w.n):
            np.testing.assert_array_equal(st.idx[i], sets[t, i])
            np.testing.assert_array_equal(np.flatnonzero(st.gi[i] != gi_old[i]), sets[t, i][grads[i][sets[t, i]] != gi_old[i][sets[t, i]]])
            np.testing.assert_allclose(st.gi[i][sets[t, i]], grads[i][sets[t, i]], rtol=1e-15)      # g_i takes the gradient's entries


def test_theory_constants_closed_forms():
    # Section 3.3 and Example 1: sqrt(beta/theta) = sqrt(1-alpha)/(1-sqrt(1-alpha)) = (1+sqrt(1-alpha))/alpha - 1.
    for alpha in (1 / 300, 4 / 64, 0.5, 0.999):
        theta = 1 - math.sqrt(1 - alpha)
        beta = (1 - alpha) / (1 - math.sqrt(1 - alpha))
        a = math.sqrt(beta / theta)
        assert a == pytest.approx(math.sqrt(1 - alpha) / (1 - math.sqrt(1 - alpha)), rel=1e-12)
        assert a == pytest.approx((1 + math.sqrt(1 - alpha)) / alpha - 1, rel=1e-9)
        assert a <= 2 / alpha - 1


@pytest.mark.parametrize("precision", ["f32", "f64"])
def test_static_input_markov_compressor_end_state(precision):
    # Section 3.1 with a constant input v^t = V_i and g_i^0 = 0: after t rounds g_i equals V_i on the
    # t*k coordinates of largest |V_i| (ties to the lower index) and 0 elsewhere -- exactly, since
    # V - 0 = V and V - V = 0 -- and the distortion ||g_i - V_i||^2 contracts by (1 - k/d) (Eq. 3).
    o = oracle_mod.Oracle(precision)
    n, d, k, T = 3, 500, 7, 20
    V = np.stack([inputs.stress_vector(11, i, d) for i in range(n)]).astype(o.real)
    st = oracle_mod.State(o, n, d, k, 0.01)
    st.init(1)
    x = np.zeros(d, dtype=np.float64)
    dist_prev = np.sum(V.astype(np.float64) ** 2, axis=1)
    for t in range(1, T + 1):
        x = x - 0.01 * st.g.astype(np.float64)
        st.step_grads(V, 1)
        for i in range(n):
            keep, vals = _brute_topk(V[i], t * k)
            expect = np.zeros(d, dtype=o.real); expect[keep] = vals
            np.testing.assert_array_equal(st.gi[i], expect)
        dist = np.sum((st.gi.astype(np.float64) - V) ** 2, axis=1)
        assert np.all(dist <= (1 - k / d) * dist_prev * (1 + 1e-12))
        dist_prev = dist
        np.testing.assert_allclose(st.g, st.gi.astype(np.float64).mean(axis=0), rtol=0,
                                   atol=1e-5 if precision == "f32" else 1e-14)
        np.testing.assert_allclose(st.x, x, rtol=0, atol=2e-6 if precision == "f32" else 1e-14)


def _fma_f32(a, b, c):
    """round_to_nearest_even_fp32(a*b + c) from exact rational arithmetic."""
    from fractions import Fraction
    q = Fraction(float(a)) * Fraction(float(b)) + Fraction(float(c))
    f = np.float32(float(q))
    cands = {float(f), float(np.nextafter(f, np.float32(np.inf))), float(np.nextafter(f, np.float32(-np.inf)))}
    best = min(cands, key=lambda t: (abs(Fraction(t) - q), int(np.float32(t).view(np.uint32)) & 1))
    return np.float32(best)


def test_fp32_state_updates_are_single_rounded_operations(oracle32):
    # The fp32 build must perform g_i + c, s*(1/n), g + p and fma(-gamma, g, x) each as one IEEE operation.
    rng = np.random.default_rng(9)
    n, d, k = 5, 40, 3
    V = rng.standard_normal((n, d)).astype(np.float32)
    st = oracle_mod.State(oracle32, n, d, k, 0.37)
    st.init_from_grads(V, mode=0)
    for _ in range(5):
        gi, g, x = st.gi.copy(), st.g.copy(), st.x.copy()
        st.step_grads(V, 1)
        x_expect = np.array([_fma_f32(-np.float32(0.37), g[j], x[j]) for j in range(d)], dtype=np.float32)
        np.testing.assert_array_equal(st.x, x_expect)
        s = np.zeros(d, dtype=np.float32); touched = np.zeros(d, dtype=bool)
        for i in range(n):
            v = V[i] - gi[i]
            keep, vals = _brute_topk(v, k)
            np.testing.assert_array_equal(st.idx[i], keep)
            np.testing.assert_array_equal(st.val[i], vals)
            for j, c in zip(keep, vals):
                gi[i, j] = np.float32(gi[i, j] + c)
                s[j] = np.float32(s[j] + c); touched[j] = True
        inv_n = np.float32(1.0) / np.float32(n)
        g_expect = np.where(touched, (g + (s * inv_n).astype(np.float32)).astype(np.float32), g)
        np.testing.assert_array_equal(st.gi, gi)
        np.testing.assert_array_equal(st.g, g_expect)


# ---------------------------------------------------------------------------
# EF21+ (Algorithm 3)
# ---------------------------------------------------------------------------

def _read_kv(path):
    out = {}
    with open(path) as fh:
        for line in fh:
            tok = line.split()
            if tok and not tok[0].startswith("#"):
                out[tok[0]] = [float(t) for t in tok[1:]]
    return out


@pytest.mark.parametrize("precision", ["f32", "f64"])
def test_alg3_hand_worked_round(precision):
    o = oracle_mod.Oracle(precision)
    kv = _read_kv(os.path.join(GOLDEN, "alg3_hand_example.txt"))
    st = oracle_mod.State(o, 2, 2, 1, 0.5)
    st.gi[:] = np.array([kv["g1"], kv["g2"]])
    st.plus_round(np.array([kv["grad1"], kv["grad2"]]))
    np.testing.assert_array_equal(st.gi, [kv["new_g1"], kv["new_g2"]])
    np.testing.assert_array_equal(st.g, kv["new_g"])
    np.testing.assert_array_equal(st.choice, kv["choice"])
    np.testing.assert_array_equal(st.idx[:, 0], kv["idx"])
    np.testing.assert_array_equal(st.val[:, 0], kv["val"])


def test_ef21_plus_takes_the_better_compressor_and_keeps_the_rate(oracle64):
    # Section 3.4: G_i^{t+1} <= min(B_i, M_i) <= M_i, so Lemma 2's bound and Theorem 1 carry over;
    # g is the plain mean of the g_i (Algorithm 3, master line).
    w = inputs.config(0)
    k = 4
    gamma = inputs.theory_gamma(w.A, w.row_offsets, w.lam, k)
    theta = 1 - math.sqrt(1 - k / w.d)
    st = oracle_mod.State(oracle64, w.n, w.d, k, gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(0)
    T = 40
    f0 = st.loss()
    _, G0 = oracle64.diagnostics(w.A, w.y, w.row_offsets, st.x, w.lam, st.gi)
    sq = []
    took_plain = 0
    for _ in range(T):
        nrm2, _ = oracle64.diagnostics(w.A, w.y, w.row_offsets, st.x, w.lam, st.gi)
        sq.append(nrm2)
        gi_old = st.gi.copy()
        st.plus_step(1)
        grads = st.grads()
        np.testing.assert_allclose(st.g, st.gi.mean(axis=0), rtol=0, atol=1e-15)
        for i in range(w.n):
            ib, vb = _brute_topk(grads[i], k)
            b = np.zeros(w.d); b[ib] = vb
            im, vm = _brute_topk(grads[i] - gi_old[i], k)
            m = gi_old[i].copy(); m[im] += vm
            B, M = np.sum((b - grads[i]) ** 2), np.sum((m - grads[i]) ** 2)
            expect = m if M <= B else b
            np.testing.assert_allclose(st.gi[i], expect, rtol=0, atol=1e-15)
            assert st.choice[i] == (0 if M <= B else 1)
            assert np.sum((st.gi[i] - grads[i]) ** 2) <= min(B, M) * (1 + 1e-12) + 1e-30
            took_plain += int(st.choice[i])
    assert np.mean(sq) <= 2 * f0 / (gamma * T) + G0 / (theta * T)


def test_ef21_plus_plain_branch_is_exercised(oracle64):
    # far-off g_i (arbitrary initialisation is allowed, Section 3.3) make C(grad) the better choice at first
    w = inputs.config(0)
    st = oracle_mod.State(oracle64, w.n, w.d, 4, 0.05, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(1)
    st.gi[:] = 3.0
    st.g[:] = 3.0
    st.plus_step(1)
    assert st.choice.sum() == w.n
    for i in range(w.n):
        assert np.count_nonzero(st.gi[i]) <= 4


# ---------------------------------------------------------------------------
# Least squares objective (Appendix A.2)
# ---------------------------------------------------------------------------

@pytest.fixture
def ls_oracle64(oracle64):
    oracle64.set_objective(1)
    yield oracle64
    oracle64.set_objective(0)


def test_least_squares_loss_and_gradient(ls_oracle64):
    # f_i = (1/m) sum (a.x - y)^2 : closed form gradient (2/m) A^T (A x - y), and central differences
    o = ls_oracle64
    w = inputs.config(0)
    rng = np.random.default_rng(8)
    x = rng.standard_normal(w.d)
    A = w.A[:50].astype(np.float64); y = w.y[:50].astype(np.float64)
    res = A @ x - y
    assert o.local_loss(w.A[:50], w.y[:50], x, 0.0) == pytest.approx(np.mean(res ** 2), rel=1e-13)
    np.testing.assert_allclose(o.local_grad(w.A[:50], w.y[:50], x, 0.0), 2.0 * A.T @ res / 50, rtol=1e-12, atol=1e-14)
    g = o.local_grad(w.A[:50], w.y[:50], x, 0.1)
    h = 1e-6
    for j in (0, 17, 63):
        e = np.zeros(w.d); e[j] = h
        fd = (o.local_loss(w.A[:50], w.y[:50], x + e, 0.1) - o.local_loss(w.A[:50], w.y[:50], x - e, 0.1)) / (2 * h)
        assert fd == pytest.approx(g[j], rel=1e-6, abs=1e-8)


def test_least_squares_ef21_converges_linearly(ls_oracle64):
    # Theorem 2 (PL case): with the stepsize bound of Eq. 16 the Lyapunov function decreases geometrically;
    # here only monotone decrease of f + (gamma/theta) G and a large overall drop are checked.
    o = ls_oracle64
    w = inputs.config(0)
    k = 8
    L_i = inputs.smoothness_constants(w.A, w.row_offsets, 0.0, "least_squares")
    L, Lt = float(np.mean(L_i)), float(np.sqrt(np.mean(L_i ** 2)))
    alpha = k / w.d
    theta = 1 - math.sqrt(1 - alpha); beta = (1 - alpha) / (1 - math.sqrt(1 - alpha))
    gamma = 1.0 / (L + Lt * math.sqrt(2 * beta / theta))
    st = oracle_mod.State(o, w.n, w.d, k, gamma, 0.0, w.A, w.y, w.row_offsets, w.x0)
    st.init(0)
    psi = []
    for _ in range(200):
        _, G = o.diagnostics(w.A, w.y, w.row_offsets, st.x, 0.0, st.gi)
        psi.append(st.loss() + gamma / theta * G)
        st.step(1)
    assert all(b <= a + 1e-12 for a, b in zip(psi, psi[1:]))
    assert psi[-1] < 0.7 * psi[0]


# ---------------------------------------------------------------------------
# Stochastic EF21 (Algorithm 5)
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("precision", ["f32", "f64"])
def test_minibatch_of_all_rows_is_the_full_step(precision):
    # tau = m_i with the rows in their own order: Algorithm 5 is Algorithm 2
    o = oracle_mod.Oracle(precision)
    w = inputs.config(0)
    m = int(np.min(np.diff(w.row_offsets)))
    assert np.all(np.diff(w.row_offsets) == m)
    a = oracle_mod.State(o, w.n, w.d, w.k, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0); a.init(0)
    b = oracle_mod.State(o, w.n, w.d, w.k, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0); b.init(0)
    batch = np.tile(np.arange(m, dtype=np.int32), (w.n, 1))
    for _ in range(5):
        a.step(1); b.step_minibatch(batch)
        for u, v in ((a.x, b.x), (a.g, b.g), (a.gi, b.gi), (a.val, b.val)):
            np.testing.assert_array_equal(u, v)
        np.testing.assert_array_equal(a.idx, b.idx)


def test_minibatch_estimate_is_the_gradient_of_the_selected_rows(oracle64):
    # From g_i = 0 and g = 0 with k = d the first message is the whole estimate, so g_i = ghat_i; it must be
    # the gradient of the sub-shard made of exactly the chosen rows (in particular: the right worker's rows)
    o = oracle64
    w = inputs.config(0)
    tau = 7
    batch = inputs.minibatch_rows(3, 0, w.row_offsets, tau)
    st = oracle_mod.State(o, w.n, w.d, w.d, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0); st.init(1)
    st.step_minibatch(batch)
    np.testing.assert_array_equal(st.x, w.x0.astype(np.float64))
    for i in range(w.n):
        rows = w.row_offsets[i] + batch[i].astype(np.int64)
        expect = o.local_grad(w.A[rows], w.y[rows], w.x0.astype(np.float64), w.lam)
        np.testing.assert_array_equal(st.gi[i], expect)
    np.testing.assert_allclose(st.g, st.gi.mean(axis=0), rtol=1e-13, atol=1e-16)


def test_minibatch_estimate_is_unbiased_over_all_subsets(oracle64):
    # Assumption of Algorithm 5's analysis: E[ghat_i] = grad f_i.  Brute force over all C(6,3) batches.
    import itertools
    o = oracle64
    rng = np.random.default_rng(21)
    m, d, tau, lam = 6, 5, 3, 0.1
    A = rng.standard_normal((m, d)).astype(np.float32)
    y = np.sign(rng.standard_normal(m)).astype(np.float32)
    x = rng.standard_normal(d)
    off = np.array([0, m], dtype=np.int64)
    acc = np.zeros(d); count = 0
    for rows in itertools.combinations(range(m), tau):
        st = oracle_mod.State(o, 1, d, d, 0.0, lam, A, y, off, x); st.init(1)
        st.step_minibatch(np.array([rows], dtype=np.int32))
        acc += st.gi[0]; count += 1
    assert count == 20
    np.testing.assert_allclose(acc / count, o.local_grad(A, y, x, lam), rtol=1e-12, atol=1e-14)


def test_minibatch_order_only_changes_rounding(oracle64):
    o = oracle64
    w = inputs.config(0)
    batch = inputs.minibatch_rows(4, 1, w.row_offsets, 16)
    a = oracle_mod.State(o, w.n, w.d, w.d, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0); a.init(1)
    b = oracle_mod.State(o, w.n, w.d, w.d, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0); b.init(1)
    a.step_minibatch(batch); b.step_minibatch(batch[:, ::-1].copy())
    np.testing.assert_allclose(a.gi, b.gi, rtol=1e-12, atol=1e-15)


# ---------------------------------------------------------------------------------------------
# EF, the original error feedback method (Algorithm 4)
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("precision", ["f32", "f64"])
def test_alg4_hand_worked_example(precision):
    o = oracle_mod.Oracle(precision)
    kv = _read_kv(os.path.join(GOLDEN, "alg4_hand_example.txt"))
    V = np.array([kv["grad1"], kv["grad2"]])
    st = oracle_mod.EFState(o, 2, 3, 1, kv["gamma"][0])
    st.init_from_grads(V)
    np.testing.assert_array_equal(st.x, 0.0)
    np.testing.assert_array_equal(st.e, 0.0)
    np.testing.assert_array_equal(st.idx[:, 0], kv["idx0"])
    np.testing.assert_array_equal(st.val[:, 0], kv["val0"])
    for t in (1, 2, 3):
        st.step_grads(V, 1)
        np.testing.assert_array_equal(st.x, kv[f"x{t}"])
        np.testing.assert_array_equal(st.e, [kv[f"e1_{t}"], kv[f"e2_{t}"]])
        np.testing.assert_array_equal(st.idx[:, 0], kv[f"idx{t}"])
        np.testing.assert_array_equal(st.val[:, 0], kv[f"val{t}"])


def test_alg4_perturbed_iterate_follows_gradient_descent(oracle64):
    # Summing Algorithm 4's error update over the nodes and adding the master line gives, for
    # xt^t = x^t - (1/n) sum_i e_i^t, the exact recursion xt^{t+1} = xt^t - gamma grad f(x^t):
    # whatever the compressor dropped stays in the errors.  The identity fails for a wrong sign, a
    # dropped term or a wrong worker/coordinate index anywhere in the loop.
    w = inputs.config(0)
    gamma = 0.05
    st = oracle_mod.EFState(oracle64, w.n, w.d, w.k, gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init()
    for _ in range(30):
        x_old, e_old = st.x.copy(), st.e.copy()
        grad_old = oracle64.all_grads(w.A, w.y, w.row_offsets, x_old, w.lam).mean(axis=0)
        idx_old, val_old = st.idx.copy(), st.val.copy()
        st.step(1)
        lhs = st.x - st.e.mean(axis=0)
        rhs = x_old - e_old.mean(axis=0) - gamma * grad_old
        np.testing.assert_allclose(lhs, rhs, rtol=0, atol=1e-14)
        # master line: x moves by the mean of the messages that were in flight
        wsum = np.zeros(w.d)
        for i in range(w.n):
            wsum[idx_old[i]] += val_old[i]
        np.testing.assert_allclose(st.x, x_old - wsum / w.n, rtol=0, atol=1e-15)
        # the new messages are Top-k of e^{t+1} + gamma grad f_i(x^{t+1}), and nothing else is sent
        grads_new = oracle64.all_grads(w.A, w.y, w.row_offsets, st.x, w.lam)
        for i in range(w.n):
            ib, vb = _brute_topk(st.e[i] + gamma * grads_new[i], w.k)
            np.testing.assert_array_equal(st.idx[i], ib)
            np.testing.assert_allclose(st.val[i], vb, rtol=0, atol=1e-15)


def test_alg4_error_is_what_the_compressor_dropped(oracle64):
    # e_i^{t+1} = (e_i^t + gamma grad f_i(x^t)) - C(e_i^t + gamma grad f_i(x^t)): zero exactly on the k kept
    # coordinates, and by Eq. 3 its squared norm is at most (1 - k/d) times that of the compressed vector.
    w = inputs.config(0)
    gamma = 0.05
    st = oracle_mod.EFState(oracle64, w.n, w.d, w.k, gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init()
    for _ in range(10):
        want = st.e + gamma * oracle64.all_grads(w.A, w.y, w.row_offsets, st.x, w.lam)
        idx = st.idx.copy()
        st.step(1)
        for i in range(w.n):
            assert np.all(st.e[i][idx[i]] == 0.0)
            rest = np.setdiff1d(np.arange(w.d), idx[i])
            np.testing.assert_allclose(st.e[i][rest], want[i][rest], rtol=0, atol=1e-16)
            assert np.sum(st.e[i] ** 2) <= (1 - w.k / w.d) * np.sum(want[i] ** 2) * (1 + 1e-12)


def test_alg4_equals_alg2_for_the_identity_compressor(oracle64):
    # Theorem 3: for a deterministic, positively homogeneous and additive compressor EF and EF21 produce
    # the same iterates.  Top-k with k = d is the identity, which is all three; both methods are then
    # gradient descent (Section 5.2) and the errors stay zero.
    w = inputs.config(0)
    gamma = 0.1
    ef = oracle_mod.EFState(oracle64, w.n, w.d, w.d, gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    ef.init()
    st = oracle_mod.State(oracle64, w.n, w.d, w.d, gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(0)
    x_gd = np.array(w.x0, dtype=np.float64)
    for _ in range(25):
        x_gd = x_gd - gamma * oracle64.all_grads(w.A, w.y, w.row_offsets, x_gd, w.lam).mean(axis=0)
        ef.step(1)
        st.step(1)
        np.testing.assert_allclose(ef.x, st.x, rtol=0, atol=1e-13)
        np.testing.assert_allclose(ef.x, x_gd, rtol=0, atol=1e-13)
        np.testing.assert_allclose(ef.e, 0.0, rtol=0, atol=1e-16)


def test_alg4_fp32_updates_are_single_rounded_operations(oracle32):
    # every update of the fp32 state is one IEEE operation: gamma*grad, e + a, (e + a) - w, s/n, x - p
    rng = np.random.default_rng(5)
    n, d, k = 3, 40, 5
    V = rng.standard_normal((n, d)).astype(np.float32)
    gamma = np.float32(0.3)
    st = oracle_mod.EFState(oracle32, n, d, k, float(gamma))
    st.init_from_grads(V)
    a = gamma * V
    np.testing.assert_array_equal(st.a, a)
    e = np.zeros((n, d), dtype=np.float32)
    x = np.zeros(d, dtype=np.float32)
    for _ in range(6):
        idx, val = st.idx.copy(), st.val.copy()
        st.step_grads(V, 1)
        s = np.zeros(d, dtype=np.float32); hit = np.zeros(d, dtype=bool)
        for i in range(n):
            for t in range(k):
                s[idx[i, t]] = np.float32(s[idx[i, t]] + val[i, t]); hit[idx[i, t]] = True
        p = (s * np.float32(np.float32(1) / np.float32(n))).astype(np.float32)
        x = np.where(hit, (x - p).astype(np.float32), x)
        for i in range(n):
            wv = np.zeros(d, dtype=np.float32); wv[idx[i]] = val[i]
            e[i] = ((e[i] + a[i]).astype(np.float32) - wv).astype(np.float32)
        np.testing.assert_array_equal(st.x.view(np.uint32), x.view(np.uint32))
        np.testing.assert_array_equal(st.e.view(np.uint32), e.view(np.uint32))
