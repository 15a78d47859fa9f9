"""GPU parity: libef21 (through its C ABI) against the CPU oracle on the same seeded inputs.

Bars: Top-k index sets and values bit-exact given identical input vectors; every state update
after the gradient bit-exact given identical gradients; local gradients within 1e-5 (relative,
norm-wise) of the oracle's fp64 gradients per step; x and f(x) within 1e-4 relative after T
iterations.
"""
import numpy as np
import pytest
import torch

import ef21_inputs as inputs
import oracle as oracle_mod
from gpu_util import (assert_state_bitwise, dev, lockstep, make_gpu, make_oracle_state, rel_l2,
                      set_gpu_state_from_oracle)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2106_05203_b200 import binding
    return binding


# ---------------------------------------------------------------------------
# Standalone Top-k
# ---------------------------------------------------------------------------

def _topk_cases():
    rng = np.random.default_rng(2024)
    cases = []
    for d, k in [(1, 1), (5, 5), (64, 4), (112, 1), (300, 16), (1000, 999), (4096, 1), (4097, 33),
                 (10007, 10), (70001, 700), (262144, 262), (300000, 299999)]:
        v = rng.standard_normal(d).astype(np.float32)
        cases.append((f"gauss-{d}-{k}", v, k))
    v = inputs.stress_vector(4, 1, 1 << 20)
    cases.append(("student-1m", v, (1 << 20) // 1000))
    v = rng.standard_normal(50000).astype(np.float32)
    v[rng.integers(0, 50000, 20000)] = np.float32(-0.75)            # many exact ties around the cut
    cases.append(("ties", v, 25000))
    cases.append(("all-equal", np.full(9000, 2.5, dtype=np.float32), 1234))
    cases.append(("all-zero", np.zeros(5000, dtype=np.float32), 7))
    v = np.zeros(6000, dtype=np.float32); v[[17, 4000, 5999]] = [1.0, -2.0, 3.0]; v[5] = -0.0
    cases.append(("fewer-nonzeros-than-k", v, 10))
    v = (rng.integers(-3, 4, 33333)).astype(np.float32) * np.float32(0.5)   # few distinct magnitudes
    cases.append(("quantised", v, 11111))
    v = rng.standard_normal(8192).astype(np.float32) * np.float32(1e-41)     # subnormals
    cases.append(("subnormal", v, 100))
    return cases


@pytest.mark.parametrize("name,v,k", _topk_cases(), ids=[c[0] for c in _topk_cases()])
def test_topk_bit_exact(name, v, k, B, oracle32):
    idx, val = B.topk(dev(v), k)
    oi, ov = oracle32.topk(v, k)
    np.testing.assert_array_equal(idx.cpu().numpy()[0], oi)
    np.testing.assert_array_equal(val.cpu().numpy()[0].view(np.uint32), ov.view(np.uint32))


def test_topk_batch_and_repeatability(B, oracle32):
    V = np.stack([inputs.stress_vector(7, i, 50001) for i in range(5)])
    idx, val = B.topk(dev(V), 50)
    idx2, val2 = B.topk(dev(V), 50)
    assert torch.equal(idx, idx2) and torch.equal(val, val2)
    for i in range(5):
        oi, ov = oracle32.topk(V[i], 50)
        np.testing.assert_array_equal(idx[i].cpu().numpy(), oi)
        np.testing.assert_array_equal(val[i].cpu().numpy(), ov)


# ---------------------------------------------------------------------------
# Local gradients (Eq. 19)
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("cfg", [0, 1, 2, 3])
def test_local_gradients_within_1e5(cfg, B, oracle32):
    w = inputs.config(cfg)
    h = make_gpu(w)
    rng = np.random.default_rng(cfg)
    for x in (w.x0, (rng.standard_normal(w.d) * 0.3).astype(np.float32)):
        h.set_x(dev(x))
        got = h.local_grads().cpu().numpy()
        want = oracle32.all_grads(w.A, w.y, w.row_offsets, x, w.lam)
        for i in range(w.n):
            assert rel_l2(got[i], want[i]) <= 1e-5, (cfg, i)
    # at x = 0 with binary features every partial sum is exact: bit-identical gradients
    if cfg in (1, 2, 3):
        h.set_x(dev(w.x0))
        got = h.local_grads().cpu().numpy()
        want = oracle32.all_grads(w.A, w.y, w.row_offsets, w.x0, w.lam)
        np.testing.assert_array_equal(got, want)


def test_local_gradients_uneven_and_empty_shards(B, oracle32):
    w = inputs.config(0)
    w.row_offsets = np.array([0, 0, 3, 150, 200], dtype=np.int64)     # an empty shard and ragged ones
    h = make_gpu(w)
    x = np.linspace(-0.5, 0.5, w.d).astype(np.float32)
    h.set_x(dev(x))
    got = h.local_grads().cpu().numpy()
    want = oracle32.all_grads(w.A, w.y, w.row_offsets, x, w.lam)
    for i in range(w.n):
        assert rel_l2(got[i], want[i]) <= 1e-5


@pytest.mark.parametrize("d", [1, 5, 127, 128, 129, 256, 300, 384, 500, 513, 700, 768, 1000, 1024, 1025, 1500])
def test_local_gradients_every_row_width(d, B, oracle32):
    # launch-per-stage gradient kernels: each register layout of the one-read kernel (up to 1,024 columns,
    # full and ragged last chunk), the two-sweep kernel beyond, ragged tiles (shards of 1, 7, 300 and 611 rows
    # and an empty one), loss and gradients
    rng = np.random.default_rng(1000 + d)
    off = np.array([0, 1, 8, 8, 308, 919], dtype=np.int64)
    n, N = len(off) - 1, int(off[-1])
    A = rng.standard_normal((N, d)).astype(np.float32) / np.float32(np.sqrt(d))
    y = np.where(rng.random(N) < 0.5, -1.0, 1.0).astype(np.float32)
    x = (rng.standard_normal(d) * 0.5).astype(np.float32)
    lam = 0.1
    h = B.EF21(n, d, 1, 0.1, lam, total_rows=N)
    h.set_path(B.PATH_LAUNCHES)
    h.load_shards(dev(A), dev(y), off)
    h.set_x(dev(x))
    got = h.local_grads().cpu().numpy()
    want = oracle32.all_grads(A, y, off, x, lam)
    for i in range(n):
        assert rel_l2(got[i], want[i]) <= 1e-5, (d, i)
    h.init(B.INIT_ZERO)
    assert h.eval()[0] == pytest.approx(oracle32.loss(A, y, off, x, lam), rel=1e-6)
    assert h.poll() == 0


@pytest.mark.parametrize("d,k", [(1, 1), (2, 1), (300, 1), (300, 300), (511, 7), (512, 512), (513, 64), (4097, 40),
                                 (8191, 8191), (8192, 1), (8192, 300), (8193, 300)])
def test_topk_short_vectors_one_launch(d, k, B, oracle32):
    # the one-launch kernel (up to 8,192 entries) and the first size beyond it, on heavy ties: quantised
    # values, blocks of equal magnitude with both signs, zeros of both signs
    rng = np.random.default_rng(d * 31 + k)
    V = (np.round(rng.standard_normal((3, d)) * 4) / 4).astype(np.float32)
    V[1, ::3] = np.float32(-0.0)
    V[2] = np.where(rng.random(d) < 0.5, np.float32(1.5), np.float32(-1.5))
    idx, val = B.topk(dev(V), k)
    idx, val = idx.cpu().numpy(), val.cpu().numpy()
    for i in range(3):
        wi, wv = oracle32.topk(V[i], k)
        np.testing.assert_array_equal(idx[i], wi)
        np.testing.assert_array_equal(val[i].view(np.uint32), wv.view(np.uint32))


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("side_stream", [False, True])
def test_launch_path_many_steps_in_one_call_equal_single_steps(variant, side_stream, B):
    # a call of several iterations replays the iteration as a graph from the second one on: same bits as
    # one call per iteration, on the default stream and on a stream of the caller's, for every method
    import torch
    w = inputs.config(2, k=4)
    outs = []
    for chunks in ((12,), (1,) * 12, (5, 1, 6)):
        stream = torch.cuda.Stream() if side_stream else None
        with torch.cuda.stream(stream) if stream is not None else torch.cuda.stream(torch.cuda.current_stream()):
            h = B.EF21(w.n, w.d, 4, w.gamma, w.lam, total_rows=w.N, stream=stream)
            h.set_path(B.PATH_LAUNCHES); h.set_variant(variant)
            h.load_shards(dev(w.A), dev(w.y), w.row_offsets)
            h.init(B.INIT_ZERO if variant == 2 else B.INIT_COMPRESSED)
            for s_ in chunks:
                h.step(s_)
            outs.append(h.get_state_host())
            assert h.poll() == 0 and h.last_path == B.PATH_LAUNCHES
    for other in outs[1:]:
        for a_, b_ in zip(outs[0], other):
            np.testing.assert_array_equal(a_, b_)


def test_launch_path_wide_rows_many_steps(B, oracle32):
    # d = 3,000: two-sweep gradient kernel, one-launch Top-k, two aggregation tiles (offsets recomputed every
    # iteration, also inside the replayed graph); a multi-step call equals single steps and tracks the oracle
    rng = np.random.default_rng(77)
    n, d, k, N = 3, 3000, 30, 600
    off = np.array([0, 150, 420, 600], dtype=np.int64)
    A = (rng.standard_normal((N, d)) / np.sqrt(d)).astype(np.float32)
    y = np.where(rng.random(N) < 0.5, -1.0, 1.0).astype(np.float32)
    outs = []
    for chunks in ((8,), (1,) * 8):
        h = B.EF21(n, d, k, 0.5, 0.1, total_rows=N)
        h.load_shards(dev(A), dev(y), off)
        h.init(B.INIT_COMPRESSED)
        for s_ in chunks:
            h.step(s_)
        assert h.last_path == B.PATH_LAUNCHES and h.poll() == 0
        outs.append(h.get_state_host())
    for a_, b_ in zip(outs[0], outs[1]):
        np.testing.assert_array_equal(a_, b_)
    st = oracle_mod.State(oracle32, n, d, k, 0.5, 0.1, A, y, off)
    st.init(0); st.step(8)
    assert rel_l2(outs[0][0], st.x) <= 1e-4


def test_eval_matches_oracle(B, oracle32):
    w = inputs.config(0)
    h = make_gpu(w); h.init(B.INIT_COMPRESSED); h.step(5)
    x, g, gi, _, _ = h.get_state_host()
    f, nrm2, G = h.eval()
    assert f == pytest.approx(oracle32.loss(w.A, w.y, w.row_offsets, x, w.lam), rel=1e-6)
    on, oG = oracle32.diagnostics(w.A, w.y, w.row_offsets, x, w.lam, gi)
    assert nrm2 == pytest.approx(on, rel=1e-4)
    assert G == pytest.approx(oG, rel=1e-4)


# ---------------------------------------------------------------------------
# Algorithm 2 with supplied gradients: everything is bit-exact
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("n,d,k,mode", [(2, 4, 1, 0), (4, 64, 4, 0), (3, 5000, 50, 1), (8, 70001, 70, 0),
                                        (5, 300, 300, 2), (20, 112, 1, 1), (1, 1, 1, 0), (64, 4097, 4, 1)])
def test_supplied_gradients_bit_exact(n, d, k, mode, B, oracle32):
    V = np.stack([inputs.stress_vector(100 + n, i, d) for i in range(n)])
    gamma = 0.01
    h = B.EF21(n, d, k, gamma)
    st = oracle_mod.State(oracle32, n, d, k, gamma)
    Vd = dev(V)
    h.init_grads(Vd, mode); st.init_from_grads(V, mode)
    assert_state_bitwise(h, st, "init")
    for t in range(6):
        h.step_grads(Vd, 1); st.step_grads(V, 1)
        assert_state_bitwise(h, st, f"step {t}")
    h.step_grads(Vd, 5); st.step_grads(V, 5)
    assert_state_bitwise(h, st, "5 steps in one call")
    assert h.poll() == 0


def test_hand_worked_example_on_gpu(B):
    # the same hand-derived run of Algorithm 2 the oracle is pinned to (tests/golden)
    from test_oracle_pins import _read_hand_example
    scal, vec = _read_hand_example()
    V = np.array([vec["V1"], vec["V2"]], dtype=np.float32)
    h = B.EF21(2, 4, 1, scal["gamma"])
    h.init_grads(dev(V), 0)
    for t in range(4):
        x, g, gi, li, lv = h.get_state_host()
        np.testing.assert_array_equal(x, vec[(f"t{t}", "x")])
        np.testing.assert_array_equal(g, vec[(f"t{t}", "g")])
        np.testing.assert_array_equal(gi[0], vec[(f"t{t}", "g1")])
        np.testing.assert_array_equal(gi[1], vec[(f"t{t}", "g2")])
        if t:
            np.testing.assert_array_equal(li[:, 0], vec[(f"t{t}", "idx")])
            np.testing.assert_array_equal(lv[:, 0], vec[(f"t{t}", "val")])
        h.step_grads(dev(V), 1)


def test_changing_supplied_gradients(B, oracle32):
    n, d, k = 6, 3001, 30
    rng = np.random.default_rng(3)
    h = B.EF21(n, d, k, 0.05); st = oracle_mod.State(oracle32, n, d, k, 0.05)
    h.init_grads(None, 1); st.init(1)
    for t in range(8):
        V = rng.standard_normal((n, d)).astype(np.float32)
        h.step_grads(dev(V), 1); st.step_grads(V, 1)
        assert_state_bitwise(h, st, f"step {t}")


# ---------------------------------------------------------------------------
# Algorithm 2 on the logistic objective
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("mode", [0, 1, 2])
def test_init_modes(mode, B, oracle32):
    w = inputs.config(1)
    h = make_gpu(w); st = make_oracle_state(oracle32, w)
    h.init(mode); st.init(mode)
    if mode == 0:
        assert_state_bitwise(h, st, "init mode 0")
    x, g, gi, _, _ = h.get_state_host()
    np.testing.assert_array_equal(gi, st.gi)      # x0 = 0 and binary features: exact
    np.testing.assert_array_equal(g, st.g)


PATHS = pytest.mark.parametrize("path", [1, 2], ids=["launches", "persistent"])


@PATHS
def test_teacher_forced_steps_tiny(path, B, oracle32):
    w = inputs.config(0)
    h = make_gpu(w, path=path); st = make_oracle_state(oracle32, w)
    h.init(0); st.init(0)
    set_gpu_state_from_oracle(h, st)
    for t in range(20):
        st_prev_gi = st.gi.copy()
        h.step(1); st.step(1)
        x, g, gi, li, lv = h.get_state_host()
        np.testing.assert_array_equal(x, st.x)                    # x update is exact given g
        np.testing.assert_array_equal(li, st.idx)
        assert np.max(np.abs(lv - st.val)) <= 1e-5 * np.max(np.abs(st.val))
        set_gpu_state_from_oracle(h, st)


@PATHS
def test_free_running_tiny_T100(path, B, oracle32):
    w = inputs.config(0)
    h = make_gpu(w, path=path); st = make_oracle_state(oracle32, w)
    h.init(0); st.init(0)
    h.step(w.T); st.step(w.T)
    assert h.last_path == path
    x, g, gi, _, _ = h.get_state_host()
    assert rel_l2(x, st.x) <= 1e-4
    # g and the g_i are not compared in a free run: the entries of grad_i - g_i that Top-k is about to take sit at
    # nearly the same magnitude (each round knocks the largest ones down), so a last-bit difference in a gradient
    # swaps the order in which two of them are sent; g_i and g then differ by one message entry (here 8e-5 on a g
    # of 1e-3 after 100 iterations, measured) until the other entry follows a round later, while x, which
    # integrates g, stays within its tolerance.  The lock-stepped tests compare g_i and g at every iteration.
    f_gpu = h.eval()[0]
    assert f_gpu == pytest.approx(st.loss(), rel=1e-4)
    assert oracle32.loss(w.A, w.y, w.row_offsets, x, w.lam) == pytest.approx(st.loss(), rel=1e-4)
    assert h.poll() == 0


@pytest.mark.parametrize("cfg", [1, 2])
def test_free_running_paper_shapes_full_T(cfg, B, oracle32):
    """The benchmark's own runs: workloads [1] and [2] (Top-1), T = 2,000 iterations in the launch configuration
    that bench.py times (automatic path and shape), against 2,000 oracle iterations: x and f(x) within 1e-4."""
    w = inputs.config(cfg)
    h = make_gpu(w); st = make_oracle_state(oracle32, w)
    h.init(0); st.init(0)
    h.step(w.T); st.step(w.T)
    assert w.T == 2000 and h.last_path == B.PATH_PERSISTENT
    x = h.get_state_host()[0]
    assert rel_l2(x, st.x) <= 1e-4
    assert h.eval()[0] == pytest.approx(st.loss(), rel=1e-4)
    assert h.poll() == 0


@PATHS
@pytest.mark.parametrize("cfg,k,steps", [(1, 1, 150), (2, 1, 40), (2, 4, 40), (2, 16, 40), (3, 1, 25)])
def test_lockstep_paper_shapes(cfg, k, steps, path, B, oracle32):
    w = inputs.config(cfg, k=k)
    h = make_gpu(w, k=k, path=path); st = make_oracle_state(oracle32, w, k=k)
    h.init(0); st.init(0)
    assert_state_bitwise(h, st, "init")
    rebased = lockstep(h, st, oracle32, w, steps, k=k)
    assert rebased <= max(2, steps // 10)
    x = h.get_state_host()[0]
    assert rel_l2(x, st.x) <= 1e-4


def test_k_equals_d_is_gradient_descent_on_gpu(B, oracle32):
    # Section 5.2: EF21 with k = d is GD; g_i tracks grad f_i to a few ulps in fp32.
    w = inputs.config(0, k=64)
    h = make_gpu(w, k=64)
    h.init(0); h.step(10)
    x, g, gi, _, _ = h.get_state_host()
    grads = h.local_grads().cpu().numpy()
    assert np.max(np.abs(gi - grads)) <= 8 * np.finfo(np.float32).eps * np.max(np.abs(grads))
    np.testing.assert_allclose(g, gi.astype(np.float64).mean(axis=0), rtol=0, atol=1e-6)


@PATHS
def test_bitwise_reproducible_and_resume(path, B):
    w = inputs.config(2, k=4)
    runs = []
    for _ in range(2):
        h = make_gpu(w, k=4, path=path); h.init(0); h.step(30)
        assert h.last_path == path
        runs.append(h.get_state_host())
    for a, b in zip(runs[0], runs[1]):
        np.testing.assert_array_equal(a, b)
    # checkpoint / resume: 15 steps, copy the state into a fresh handle, 15 more
    h1 = make_gpu(w, k=4, path=path); h1.init(0); h1.step(15)
    x, g, gi, _, _ = h1.get_state()
    h2 = make_gpu(w, k=4, path=path); h2.set_state(x, g, gi); h2.step(15)
    for a, b in zip(h2.get_state_host(messages=False)[:3], runs[0][:3]):
        np.testing.assert_array_equal(a, b)


# ---------------------------------------------------------------------------
# Persistent kernel: every launch shape, ragged shards, the bounded wait
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("src", [0, 1, 2], ids=["regs", "smem", "gmem"])
@pytest.mark.parametrize("rb", [8, 16, 32])
@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
def test_persistent_shapes_tiny(cluster, rb, src, B, oracle32):
    w = inputs.config(0)
    h = make_gpu(w, path=2)
    h.set_persistent_shape(cluster, rb, src)
    st = make_oracle_state(oracle32, w)
    h.init(0); st.init(0)
    rows_cta = -(-50 // cluster)
    if src == 0 and -(-rows_cta // rb) > 8:
        with pytest.raises(B.Ef21Error) as e:
            h.step(1)
        assert e.value.status == 7
        return
    assert lockstep(h, st, oracle32, w, 12) == 0
    assert h.get_persistent_shape() == (cluster, rb, src)
    assert h.poll() == 0


@pytest.mark.parametrize("d,k,cluster", [(1, 1, 1), (5, 2, 2), (130, 3, 4), (257, 8, 8), (300, 32, 3), (511, 5, 7)])
def test_persistent_dimensions_and_ragged_shards(d, k, cluster, B, oracle32):
    n, N = 5, 333
    w = inputs.make_logistic("ragged", n=n, d=d, N=N, k=k, seed=d, features="gauss", flip=0.1, gamma=0.05, T=10)
    w.row_offsets = np.array([0, 0, 7, 100, 290, 333], dtype=np.int64)
    h = make_gpu(w, path=2)
    h.set_persistent_shape(cluster, 0, -1)
    st = make_oracle_state(oracle32, w)
    h.init(0); st.init(0)
    try:
        h.step(1)
    except B.Ef21Error as e:               # a cluster size this device cannot co-schedule
        assert e.status == 7 and cluster in (3, 7)
        return
    st.step(1)
    assert lockstep(h, st, oracle32, w, 10) <= 1
    assert h.poll() == 0


@pytest.mark.parametrize("d,rb,threads,src", [(64, 4, 512, 1), (64, 16, 512, 0), (200, 8, 512, 2), (300, 4, 512, 1),
                                              (300, 4, 256, 2), (120, 8, 512, 0), (500, 8, 256, 1)])
def test_persistent_block_sizes(d, rb, threads, src, B, oracle32):
    w = inputs.make_logistic("blocks", n=6, d=d, N=900, k=2, seed=1000 + d, features="gauss", flip=0.1, gamma=0.05, T=10)
    h = make_gpu(w, path=2)
    h.set_persistent_shape(2, rb, src)
    h.set_persistent_threads(threads)
    st = make_oracle_state(oracle32, w)
    h.init(0); st.init(0)
    assert lockstep(h, st, oracle32, w, 10) <= 1
    assert h.get_persistent_shape() == (2, rb, src) and h.get_persistent_threads() == threads
    assert h.poll() == 0


@pytest.mark.parametrize("body", [1, 2], ids=["serving-warp", "whole-block"])
@pytest.mark.parametrize("cfg,k,steps", [(0, 4, 30), (0, 1, 30), (1, 1, 60), (2, 4, 20), (3, 1, 15)])
def test_persistent_bodies_track_the_oracle(cfg, k, steps, body, B, oracle32):
    # both bodies of the persistent kernel on every kind of shape (rows in registers, one extra row per warp, rows
    # from global memory; one and several polling rounds), iteration by iteration against the oracle
    w = inputs.config(cfg, k=k)
    h = make_gpu(w, k=k, path=2); h.set_persistent_body(body)
    st = make_oracle_state(oracle32, w, k=k)
    h.init(0); st.init(0)
    lockstep(h, st, oracle32, w, steps, k=k)
    assert h.last_path == B.PATH_PERSISTENT and h.get_persistent_body() == body
    # several iterations in one launch give the same bits as the same iterations one launch each
    outs = []
    for chunks in ((7,), (1,) * 7):
        h2 = make_gpu(w, k=k, path=2); h2.set_persistent_body(body); h2.init(0)
        for s_ in chunks:
            h2.step(s_)
        outs.append(h2.get_state_host())
    for a_, b_ in zip(outs[0], outs[1]):
        np.testing.assert_array_equal(a_, b_)
    assert h.poll() == 0 and h2.poll() == 0


def test_persistent_body_choice(B):
    w = inputs.config(0, k=1)
    h = make_gpu(w, k=1, path=2); h.init(0); h.step(2)
    assert h.get_persistent_body() == 1                 # Top-1: the serving-warp body
    w = inputs.config(0, k=4)
    h = make_gpu(w, k=4, path=2); h.init(0); h.step(2)
    assert h.get_persistent_body() == 2                 # several entries per message: whole-block steps
    w = inputs.config(0, k=16)
    h = make_gpu(w, k=16, path=2); h.set_persistent_body(1); h.init(0)
    with pytest.raises(B.Ef21Error) as e:
        h.step(1)                                       # the serving-warp body stops at k = 8
    assert e.value.status == 7


@pytest.mark.parametrize("body", [1, 2], ids=["serving-warp", "whole-block"])
def test_persistent_epochs_wrap_around(body, B, oracle32):
    # the 16-bit epoch of the message words runs on from launch to launch and wraps from 65,535 to 1: a run that
    # crosses the wrap inside a launch, and one that crosses it between launches, give the same bits
    w = inputs.config(0, k=2)
    outs = []
    for chunks in ((65500, 200), (65535, 1, 164), (30000, 35700)):
        h = make_gpu(w, k=2, path=2); h.set_persistent_body(body); h.init(0)
        for s_ in chunks:
            h.step(s_)
        assert h.poll() == 0
        outs.append(h.get_state_host())
    for other in outs[1:]:
        for a_, b_ in zip(outs[0], other):
            np.testing.assert_array_equal(a_, b_)
    assert np.all(np.isfinite(outs[0][0]))
    # long after convergence the iterate is a stationary point of the oracle's objective as well
    grads = oracle32.all_grads(w.A, w.y, w.row_offsets, outs[0][0], w.lam).astype(np.float64)
    assert np.linalg.norm(grads.mean(axis=0)) <= 1e-4


def test_two_handles_share_the_kernels(B, oracle32):
    # two handles of different shapes take turns on one stream: each keeps its own cached launch plan, message slots
    # and epochs, and both follow the oracle
    wa, wb = inputs.config(0, k=1), inputs.config(1)
    ha, hb = make_gpu(wa, k=1, path=2), make_gpu(wb, path=2)
    sa, sb = make_oracle_state(oracle32, wa, k=1), make_oracle_state(oracle32, wb)
    ha.init(0); hb.init(0); sa.init(0); sb.init(0)
    for _ in range(4):
        ha.step(7); hb.step(5); sa.step(7); sb.step(5)
    assert rel_l2(ha.get_state_host()[0], sa.x) <= 1e-4
    assert rel_l2(hb.get_state_host()[0], sb.x) <= 1e-4
    assert ha.poll() == 0 and hb.poll() == 0


@pytest.mark.parametrize("body", [1, 2], ids=["serving-warp", "whole-block"])
@pytest.mark.parametrize("n,groups", [(5, 1), (20, 1), (32, 1), (20, 2), (24, 3)])
def test_workers_naming_the_same_coordinate(n, groups, body, B, oracle32):
    # `groups` distinct shards, each held by n / groups workers: in every iteration whole groups of workers send the same
    # coordinate, so the per-coordinate sums in worker order have up to n terms (all 32 lanes of a polling round for
    # n = 32; two or three interleaved groups of 8 to 10 otherwise)
    m = 40
    base = inputs.make_logistic("crowd", n=groups, d=96, N=groups * m, k=1, seed=7000 + n, features="gauss", flip=0.1, gamma=0.05, T=10)
    w = inputs.make_logistic("crowd", n=n, d=96, N=n * m, k=1, seed=7000 + n, features="gauss", flip=0.1, gamma=0.05, T=10)
    for i in range(n):
        src = i % groups
        w.A[i * m:(i + 1) * m] = base.A[src * m:(src + 1) * m]
        w.y[i * m:(i + 1) * m] = base.y[src * m:(src + 1) * m]
    h = make_gpu(w, k=1, path=2); h.set_persistent_body(body)
    st = make_oracle_state(oracle32, w, k=1)
    h.init(0); st.init(0)
    sizes = []
    for _ in range(12):
        lockstep(h, st, oracle32, w, 1, k=1)
        sizes.append(int(np.max(np.unique(st.idx[:, 0], return_counts=True)[1])))
    assert min(sizes) >= n // groups, sizes
    assert h.last_path == B.PATH_PERSISTENT and h.get_persistent_body() == body and h.poll() == 0


def test_two_handles_on_two_streams_are_kept_apart(B):
    # 120 blocks each on 148 SMs: the two launches cannot be resident together, and each needs all of its clusters at
    # once.  The library orders a persistent launch after the device's previous one when the streams differ, so both
    # run to the end and give the bits of a run alone.
    w = inputs.config(2, k=1)
    alone = make_gpu(w, k=1, path=2); alone.init(0); alone.step(400)
    want = alone.get_state_host()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    hs = []
    A_t, y_t, x_t = dev(w.A), dev(w.y), dev(w.x0)          # alive until the end of the test: the handles read them on their streams
    torch.cuda.synchronize()
    for s in (s1, s2):
        h = B.EF21(w.n, w.d, 1, w.gamma, w.lam, total_rows=w.N, stream=s)
        h.set_path(2)
        h.load_shards(A_t, y_t, w.row_offsets); h.set_x(x_t); h.init(0)
        hs.append(h)
    torch.cuda.synchronize()
    for _ in range(4):                     # no host synchronisation between the calls: the launches queue up
        hs[0].step(100); hs[1].step(100)
    for h in hs:
        assert h.poll() == 0 and h.last_path == B.PATH_PERSISTENT
        for u, v in zip(h.get_state_host(), want):
            np.testing.assert_array_equal(u, v)
    hs[1].close()                          # the last launch was this handle's: its stream must not be touched again
    hs[0].step(5)
    assert hs[0].poll() == 0


def test_persistent_many_steps_in_one_launch_equals_single_steps(B):
    w = inputs.config(1)
    a = make_gpu(w, path=2); a.init(0); a.step(300)
    b = make_gpu(w, path=2); b.init(0)
    for _ in range(30):
        b.step(10)
    for u, v in zip(a.get_state_host(), b.get_state_host()):
        np.testing.assert_array_equal(u, v)


def test_bounded_wait_times_out_and_context_survives(B):
    w = inputs.config(0)
    h = make_gpu(w, path=2); h.init(0)
    h.selftest_bounded_wait(1000)          # spins on a word nobody writes
    assert h.poll() == 5                   # EF21_ERR_TIMEOUT
    h.clear_status()
    assert h.poll() == 0
    h.step(3)                              # the device and the handle are still usable
    assert h.poll() == 0


def test_state_after_timeout_is_restored_with_set_state(B, oracle32):
    # the documented way out of EF21_ERR_TIMEOUT: the state counts as unspecified, the caller restores it with
    # ef21_set_state, clears the status word and carries on; the run then follows the oracle again
    w = inputs.config(0)
    h = make_gpu(w, path=2); st = make_oracle_state(oracle32, w)
    h.init(0); st.init(0)
    h.step(5); st.step(5)
    saved = h.get_state()[:3]
    h.selftest_bounded_wait(2000)
    assert h.poll() == 5
    h.set_state(*saved)
    h.clear_status()
    assert h.poll() == 0
    h.step(15); st.step(15)
    assert h.last_path == B.PATH_PERSISTENT
    assert rel_l2(h.get_state_host()[0], st.x) <= 1e-4
    assert h.poll() == 0


def test_non_finite_supplied_gradient_is_reported(B):
    # Section 2.1 defines the compressor on real vectors: a NaN or Inf anywhere in a compressed vector is selected
    # (largest key) and recorded as EF21_ERR_NONFINITE; the device and the handle stay usable
    for d, k in ((3000, 30), (70001, 70), (300000, 300)):          # one-launch, multi-pass and one-pass Top-k
        n = 3
        rng = np.random.default_rng(d)
        V = rng.standard_normal((n, d)).astype(np.float32)
        h = B.EF21(n, d, k, 0.01)
        h.init_grads(None, B.INIT_ZERO)
        h.step_grads(dev(V), 1)
        assert h.poll() == 0
        saved = h.get_state()[:3]
        bad = V.copy(); bad[1, d // 2] = np.nan
        h.step_grads(dev(bad), 1)
        assert h.poll() == 6, (d, "NaN")
        h.clear_status(); h.set_state(*saved)
        bad = V.copy(); bad[2, d - 1] = -np.inf
        h.step_grads(dev(bad), 1)
        assert h.poll() == 6, (d, "Inf")
        h.clear_status(); h.set_state(*saved)
        h.step_grads(dev(V), 1)
        assert h.poll() == 0


@PATHS
def test_non_finite_iterate_is_reported(path, B):
    w = inputs.config(0)
    h = make_gpu(w, path=path); h.init(0)
    h.step(3)
    assert h.poll() == 0
    saved = h.get_state()[:3]
    x = saved[0].clone(); x[7] = float("nan")
    h.set_state(x, saved[1], saved[2])
    h.step(2)
    assert h.poll() == 6
    with pytest.raises(B.Ef21Error) as e:
        h.eval()
    assert e.value.status == 6
    h.clear_status(); h.set_state(*saved)
    h.step(2)
    assert h.poll() == 0 and np.all(np.isfinite(h.get_state_host()[0]))


def test_reloading_shards_with_another_split_drops_the_captured_iteration(B, oracle32):
    # the launch path replays an iteration as a CUDA graph whose gradient grid is the number of row tiles; another
    # split of the same rows changes that number, so the graph must be captured again
    rng = np.random.default_rng(8)
    n, d, N, k = 6, 40, 6000, 3
    A = rng.standard_normal((N, d)).astype(np.float32)
    y = np.where(rng.random(N) < 0.5, -1.0, 1.0).astype(np.float32)
    even = inputs.shard_offsets(N, n)
    uneven = np.array([0, 10, 25, 3000, 3001, 5990, N], dtype=np.int64)
    h = B.EF21(n, d, k, 0.3, 0.1, total_rows=N); h.set_path(B.PATH_LAUNCHES)
    h.load_shards(dev(A), dev(y), even)
    h.init(B.INIT_COMPRESSED)
    h.step(5)                                        # captures and replays the iteration for the even split
    h.load_shards(dev(A), dev(y), uneven)
    h.set_x(dev(np.zeros(d, dtype=np.float32)))
    h.init(B.INIT_COMPRESSED)
    h.step(5)
    multi = h.get_state_host()
    h2 = B.EF21(n, d, k, 0.3, 0.1, total_rows=N); h2.set_path(B.PATH_LAUNCHES)
    h2.load_shards(dev(A), dev(y), uneven)
    h2.init(B.INIT_COMPRESSED)
    for _ in range(5):
        h2.step(1)
    for a_, b_ in zip(multi, h2.get_state_host()):
        np.testing.assert_array_equal(a_, b_)
    st = oracle_mod.State(oracle32, n, d, k, 0.3, 0.1, A, y, uneven)
    st.init(0); st.step(5)
    assert rel_l2(multi[0], st.x) <= 1e-4
    assert h.poll() == 0


def test_call_order_and_argument_errors(B):
    w = inputs.config(0)
    h = B.EF21(w.n, w.d, w.k, w.gamma, w.lam, total_rows=w.N)
    with pytest.raises(B.Ef21Error) as e:
        h.step(1)
    assert e.value.status == 2
    with pytest.raises(B.Ef21Error) as e:
        h.init(0)                       # shards not loaded
    assert e.value.status == 2
    bad = w.row_offsets.copy(); bad[-1] -= 1
    with pytest.raises(B.Ef21Error) as e:
        h.load_shards(dev(w.A), dev(w.y), bad)
    assert e.value.status == 1
    h.load_shards(dev(w.A), dev(w.y), w.row_offsets)
    with pytest.raises(B.Ef21Error):
        h.step(1)                       # not initialised
    h.init(1); h.step(1)
    assert h.poll() == 0
    with pytest.raises(B.Ef21Error):
        B.EF21(4, 64, 65, 0.1)          # k > d
