"""GPU parity for the very calls the benchmark times, at the benchmark's sizes and in its launch configuration
(automatic path and shape), each against the CPU oracle or against a property the method fixes at any size:

  * 2,000 free-running iterations of Algorithm 2 on the w8a-shaped workload (Top-1) and on the a9a-shaped one with
    k = 4 and k = 16: x within 1e-4 of the oracle's after every 100 iterations, else that stretch again iteration by
    iteration with every differing index shown to be a near-tie; x and f(x) at the end;
  * the supplied-gradient workload (n = 64, d = 4,194,304, k = 4,194) through ONE call of 50 steps: the closed-form
    end state of the Markov compressor on a static input (Section 3.1, Eqs. 9-10) on all 64 workers, and the last
    messages and g_i of sampled workers bit for bit against 50 oracle steps;
  * several steps in one call on long Student-t vectors (the second-stream path with the threshold estimated ahead),
    bit for bit;
  * shards larger than L2 (600 MB), iteration by iteration;
  * the lines for Algorithms 3 and 4 (EF21+ and EF on the mushrooms-shaped workload, 500 iterations, persistent kernels).
"""
import numpy as np
import pytest
import torch

import ef21_inputs as inputs
import oracle as oracle_mod
from gpu_util import assert_state_bitwise, dev, lockstep, make_gpu, make_oracle_state, rel_l2, set_gpu_state_from_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2106_05203_b200 import binding
    return binding


def _snapshot(st):
    return tuple(a.copy() for a in (st.x, st.g, st.gi, st.idx, st.val))


def _restore(st, snap):
    for dst, src in zip((st.x, st.g, st.gi, st.idx, st.val), snap):
        dst[...] = src


def free_run_with_rebase(h, st, o, w, k, T, chunk=100):
    """T iterations on both sides, `chunk` at a time in one call each (free-running); after every chunk x must be
    within 1e-4 of the oracle's (the bar stated for the end of the run, applied all along it).

    Top-k is discontinuous.  Once g is small, the entries of grad_i - g_i that compete for the next message differ by
    less than the last bits of a gradient, the two sides send them in a different order, and with Top-1 of 300
    coordinates the swapped entry may wait hundreds of iterations for its turn: x then parts by more than 1e-4 for
    ANY two implementations whose gradients are not bit-identical (the oracle with fp64 state against the oracle with
    fp32 state parts by up to 3e-3 within 100 iterations on the w8a-shaped workload from iteration 1,100 on).  Such a
    chunk is taken again from the oracle's state at its start, one iteration at a time (gpu_util.lockstep): every
    message must equal the oracle's, or differ at a near-tie within the per-step gradient tolerance, after which the
    GPU continues from the oracle's state.  Returns (chunks taken again, near-ties met in them)."""
    replayed, near_ties, done = [], 0, 0
    while done < T:
        s = min(chunk, T - done)
        snap = _snapshot(st)
        h.step(s); st.step(s)
        x = h.get_state_host()[0]
        if not rel_l2(x, st.x) <= 1e-4:
            replayed.append(done)
            _restore(st, snap)
            set_gpu_state_from_oracle(h, st)
            near_ties += lockstep(h, st, o, w, s, k=k)
            set_gpu_state_from_oracle(h, st)
        done += s
    return replayed, near_ties


@pytest.mark.parametrize("cfg,k", [(3, 1), (2, 4), (2, 16)])
def test_free_running_full_T_on_the_other_benchmark_shapes(cfg, k, B, oracle32):
    w = inputs.config(cfg, k=k)
    h = make_gpu(w, k=k); st = make_oracle_state(oracle32, w, k=k)
    h.init(0); st.init(0)
    replayed, near_ties = free_run_with_rebase(h, st, oracle32, w, k, w.T)
    print(f"configs[{cfg}] Top-{k}: chunks taken again from the oracle's state: {replayed}, near-ties in them: {near_ties}")
    assert w.T == 2000 and h.last_path == B.PATH_PERSISTENT
    x = h.get_state_host()[0]
    assert rel_l2(x, st.x) <= 1e-4
    assert h.eval()[0] == pytest.approx(st.loss(), rel=1e-4)
    assert replayed == [] or near_ties >= 1, "a chunk that parted must contain a near-tie that explains it"
    assert h.poll() == 0


def _capture_order(v, count):
    """Indices of the `count` entries of largest |v| in the order Top-k takes them: magnitude (bit pattern)
    descending, index ascending among equals."""
    key = v.view(np.uint32) & np.uint32(0x7FFFFFFF)
    d = key.shape[0]
    kth = np.partition(key, d - count)[d - count]
    above = np.flatnonzero(key > kth)
    equal = np.flatnonzero(key == kth)[: count - above.shape[0]]          # flatnonzero is ascending: lower index first
    cand = np.concatenate([above, equal])
    order = np.lexsort((cand, -key[cand].astype(np.int64)))
    return cand[order]


def test_stress_workload_one_call_of_50_steps(B, oracle32):
    """Section 3.1: on a static input v and from M = 0 the Markov compressor with Top-k has, after t steps, captured
    exactly the t*k entries of largest |v| (ties to the lower index) and holds v there and 0 elsewhere.  The master
    state follows in closed form: g^t is the mean of the g_i^t, and x^T = -gamma * sum_{t<T} g^t, i.e. an entry
    captured at step c contributes (T - c) times."""
    w = inputs.config(4)
    T = w.T
    assert (w.n, w.d, w.k, T) == (64, 4194304, 4194, 50)
    sampled = (5, 40, 63)
    V = torch.empty((w.n, w.d), dtype=torch.float32, device="cuda")
    h = B.EF21(w.n, w.d, w.k, w.gamma)
    h.init_grads(None, B.INIT_ZERO)
    g_expect = np.zeros(w.d, dtype=np.float64)
    x_expect = np.zeros(w.d, dtype=np.float64)
    host, orders = {}, []
    for i in range(w.n):
        vi = w.worker_vector(i)
        V[i].copy_(torch.from_numpy(vi))
        order = _capture_order(vi, T * w.k)
        orders.append(order)
        step_of = 1 + np.arange(T * w.k) // w.k                       # the step at which the entry is captured
        np.add.at(g_expect, order, vi[order].astype(np.float64))
        np.add.at(x_expect, order, vi[order].astype(np.float64) * (T - step_of))
        if i in sampled:
            host[i] = vi
    g_expect /= w.n
    x_expect *= -w.gamma / w.n
    h.step_grads(V, T)                                                # the call the benchmark times
    x, g, gi, li, lv = h.get_state()
    assert h.fallback_count() == 0 and h.poll() == 0
    for i in range(w.n):
        row = gi[i].cpu().numpy()
        nz = np.flatnonzero(row)
        np.testing.assert_array_equal(nz, np.sort(orders[i]), err_msg=f"worker {i}: captured set")
        vi = V[i].cpu().numpy()
        np.testing.assert_array_equal(row[nz].view(np.uint32), vi[nz].view(np.uint32), err_msg=f"worker {i}: values")
        np.testing.assert_array_equal(li[i].cpu().numpy(), np.sort(orders[i][(T - 1) * w.k:]), err_msg=f"worker {i}: last message")
    assert np.max(np.abs(g.cpu().numpy() - g_expect)) <= 1e-5 * np.max(np.abs(g_expect))
    assert np.max(np.abs(x.cpu().numpy() - x_expect)) <= 1e-5 * np.max(np.abs(x_expect))
    for i in sampled:
        solo = oracle_mod.State(oracle32, 1, w.d, w.k, w.gamma)
        solo.step_grads(host[i][None, :], T)
        np.testing.assert_array_equal(li[i].cpu().numpy(), solo.idx[0])
        np.testing.assert_array_equal(lv[i].cpu().numpy().view(np.uint32), solo.val[0].view(np.uint32))
        np.testing.assert_array_equal(gi[i].cpu().numpy().view(np.uint32), solo.gi[0].view(np.uint32))


@pytest.mark.parametrize("n,d,k,steps", [(8, 300000, 300, 6), (5, 1 << 20, 1048, 4)])
def test_several_steps_in_one_call_long_vectors_bit_exact(n, d, k, steps, B, oracle32):
    # the threshold of round t+1 is estimated while round t aggregates on a second stream; on Student-t input the
    # threshold hits every time, so this is the path the stress benchmark runs, here against the oracle on all state
    V = np.stack([inputs.stress_vector(300 + n, i, d) for i in range(n)])
    h = B.EF21(n, d, k, 0.01); st = oracle_mod.State(oracle32, n, d, k, 0.01)
    h.init_grads(None, B.INIT_ZERO); st.init(1)
    h.step_grads(dev(V), steps); st.step_grads(V, steps)
    assert_state_bitwise(h, st, f"{steps} steps in one call")
    h.step_grads(dev(V), 2); st.step_grads(V, 2)                     # a second call continues from the first
    assert_state_bitwise(h, st, "two more")
    assert h.fallback_count() == 0 and h.poll() == 0


@pytest.mark.parametrize("path", [0, 1], ids=["auto", "launches"])
def test_lockstep_shards_beyond_l2(path, B, oracle32):
    # 600 MB of shards: every iteration really streams the rows from HBM (global-memory row source of the
    # persistent kernel on the automatic path, the one-read gradient kernel on the launch path)
    w = inputs.hbm_scale_logistic()
    assert 4 * w.N * w.d > 4 * 126e6
    h = make_gpu(w, path=path); st = make_oracle_state(oracle32, w)
    h.init(0); st.init(0)
    assert_state_bitwise(h, st, "init (x0 = 0, binary features: exact)")
    lockstep(h, st, oracle32, w, 5)
    if path == 0:
        assert h.last_path == B.PATH_PERSISTENT and h.get_persistent_shape()[2] == 2      # rows from global memory
    got = h.local_grads().cpu().numpy()
    want = st.grads()
    for i in range(w.n):
        assert rel_l2(got[i], want[i]) <= 1e-5
    assert h.poll() == 0


@pytest.mark.parametrize("variant", ["ef21_plus", "ef"])
def test_variant_calls_of_the_benchmark(variant, B, oracle32, oracle64):
    """The benchmark's lines for Algorithms 3 and 4 on the mushrooms-shaped workload, automatic path (the persistent kernel
    of the variant), from the variant's own start: 500 iterations, free-running, 50 per call.

    After every call x must be within 1e-4 of the oracle's.  Top-k makes the trajectory discontinuous: the oracle with
    its state in fp64 parts from the oracle with its state in fp32 by 6e-4 around iteration 250 of the EF21+ run and comes
    back to 1e-4 by iteration 500 (rounding differences of 1e-7 in the state decide a near-tie some iterations later).
    Where the two oracles, running freely from one state, have parted by more than 1e-5, fp32 arithmetic cannot decide
    the trajectory; there, and only there, the GPU may part too (by no more than ten times as much), and all three
    continue from the fp32 oracle's state."""
    w = inputs.config(1)
    h = make_gpu(w)
    if variant == "ef21_plus":
        h.set_variant(B.VARIANT_EF21_PLUS)
        st, wide = make_oracle_state(oracle32, w), make_oracle_state(oracle64, w)
        h.init(0); st.init(0); wide.init(0)
        fields = ("x", "g", "gi")
        advance = lambda s_, n_: s_.plus_step(n_)
        rebase = lambda: set_gpu_state_from_oracle(h, st)
    else:
        h.set_variant(B.VARIANT_EF)
        st = oracle_mod.EFState(oracle32, w.n, w.d, w.k, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
        wide = oracle_mod.EFState(oracle64, w.n, w.d, w.k, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
        h.init(B.INIT_ZERO); st.init(); wide.init()
        fields = ("x", "e")
        advance = lambda s_, n_: s_.step(n_)
        rebase = lambda: h.set_state(dev(st.x), None, dev(st.e))
    undecidable = []
    for done in range(0, 500, 50):
        h.step(50); advance(st, 50); advance(wide, 50)
        assert h.last_path == B.PATH_PERSISTENT
        parted = rel_l2(h.get_state_host()[0], st.x)
        if parted > 1e-4:
            between_oracles = rel_l2(wide.x, st.x)
            assert between_oracles > 1e-5 and parted <= 10 * between_oracles, (done, parted, between_oracles)
            undecidable.append(done)
            rebase()
            for f in fields:                      # all three continue from one state
                getattr(wide, f)[...] = getattr(st, f)
    print(f"{variant}: stretches the arithmetic cannot decide: {undecidable}")
    assert len(undecidable) <= 3
    assert rel_l2(h.get_state_host()[0], st.x) <= 1e-4
    assert h.eval()[0] == pytest.approx(st.loss(), rel=1e-4)
    assert h.poll() == 0
