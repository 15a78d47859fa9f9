"""Helpers shared by the GPU parity tests (comparison logic only; no method arithmetic)."""
import numpy as np
import torch

import oracle as oracle_mod


def dev(a, dtype=torch.float32):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype).cuda().contiguous()


def make_gpu(w, total_rows=None, k=None, path=None):
    """EF21 handle for a LogisticWorkload with shards loaded and x0 set."""
    from paper_2106_05203_b200 import binding
    h = binding.EF21(w.n, w.d, k or w.k, w.gamma, w.lam, total_rows=w.N)
    if path is not None:
        h.set_path(path)
    h.load_shards(dev(w.A), dev(w.y), w.row_offsets)
    h.set_x(dev(w.x0))
    return h


def make_oracle_state(o, w, k=None):
    return oracle_mod.State(o, w.n, w.d, k or w.k, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return np.linalg.norm(a - b) / den if den > 0 else np.linalg.norm(a - b)


def assert_state_bitwise(h, st, what=""):
    x, g, gi, li, lv = h.get_state_host()
    np.testing.assert_array_equal(li, st.idx, err_msg=f"{what}: message indices")
    np.testing.assert_array_equal(lv.view(np.uint32), st.val.view(np.uint32), err_msg=f"{what}: message values")
    np.testing.assert_array_equal(gi.view(np.uint32), st.gi.view(np.uint32), err_msg=f"{what}: g_i")
    np.testing.assert_array_equal(g.view(np.uint32), st.g.view(np.uint32), err_msg=f"{what}: g")
    np.testing.assert_array_equal(x.view(np.uint32), st.x.view(np.uint32), err_msg=f"{what}: x")


def set_gpu_state_from_oracle(h, st):
    h.set_state(dev(st.x), dev(st.g), dev(st.gi))


def lockstep(h, st, o, w, steps, k=None, grad_tol=1e-5, advance=None, grads_of=None):
    """Advance GPU and oracle one iteration at a time from a common state.

    Every step: the GPU's messages must equal the oracle's (indices and, up to the gradient
    tolerance, values).  Where an index differs, both choices must be valid Top-k picks of vectors
    that agree within the gradient tolerance (a near-tie); the GPU is then re-based onto the
    oracle's state.  Returns the number of re-basings.

    Tolerances.  tol_i = grad_tol * max_j |grad f_i(x)_j|: the per-step bar on the local gradients
    (1e-5, stated norm-wise) applied coordinate by coordinate against the max-norm, which is never
    looser than the norm-wise bar since max|.| <= ||.||_2.  A message value may differ by tol_i.  An
    index that only one side selected must lie within 2 tol_i of the k-th magnitude: two vectors that
    agree within tol_i per entry can order two entries differently only if their magnitudes are
    within 2 tol_i of each other (one moves up, the other down).

    advance(t) (optional) performs iteration t on both sides instead of the plain step; grads_of(t)
    then returns the vectors that iteration fed to the compressor (default: the full gradients)."""
    k = k or w.k
    rebased = 0
    for t in range(steps):
        gi_old = st.gi.copy()
        if advance is None:
            h.step(1)
            st.step(1)
        else:
            advance(t)
        x, g, gi, li, lv = h.get_state_host()
        grads = (st.grads() if grads_of is None else grads_of(t)).astype(np.float64)
        scale = np.max(np.abs(grads), axis=1) + 1e-30
        dispute = False
        for i in range(w.n):
            if np.array_equal(li[i], st.idx[i]):
                assert np.max(np.abs(lv[i].astype(np.float64) - st.val[i])) <= grad_tol * scale[i], (t, i)
                continue
            dispute = True
            v = grads[i] - gi_old[i]
            kth = np.sort(np.abs(v))[::-1][k - 1]
            for j in set(li[i].tolist()) ^ set(st.idx[i].tolist()):
                assert abs(abs(v[j]) - kth) <= 2 * grad_tol * scale[i], \
                    f"step {t} worker {i}: index {j} is not a near-tie (|v|={abs(v[j])}, kth={kth})"
        if dispute:
            rebased += 1
            set_gpu_state_from_oracle(h, st)
        else:
            assert rel_l2(x, st.x) <= 1e-4 or np.linalg.norm(st.x) == 0, t
    return rebased
