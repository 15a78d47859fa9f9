"""ef21_topk_static -- Top-k for callers that must not use the CUDA allocator (a thread that cannot
afford cudaMalloc's implicit synchronisation, a plug-in in a framework that owns all device
memory, a process with a fixed memory carve-up).  Its scratch is a fixed array inside the library,
so the test checks, through the C ABI, that it gives exactly what ef21_topk gives with a
caller-provided workspace and what the CPU oracle's full-sort Top-k gives, twice in a row (the
shared scratch keeps the previous call's contents), and that sizes beyond the built-in scratch
are refused.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import ef21_inputs as inputs

pytestmark = pytest.mark.gpu


def test_topk_static_matches_topk_twice_in_a_row(oracle32):
    from paper_2106_05203_b200 import binding as B
    rng = np.random.default_rng(11)
    first = np.stack([inputs.stress_vector(21, i, 100003) for i in range(7)])
    second = rng.standard_normal((3, 9001)).astype(np.float32)
    second[:, rng.integers(0, 9001, 3000)] = np.float32(0.5)            # ties across the cut
    for V, k in ((first, 100), (second, 4000)):                         # two calls, different shapes
        v = torch.as_tensor(V).cuda()
        idx = torch.full((V.shape[0], k), -1, dtype=torch.int32, device="cuda")
        val = torch.full((V.shape[0], k), float("nan"), dtype=torch.float32, device="cuda")
        B.topk_static(v, k, idx, val)
        want_idx, want_val = B.topk(v, k)
        torch.cuda.synchronize()
        assert torch.equal(idx, want_idx)
        assert torch.equal(val.view(torch.int32), want_val.view(torch.int32))
        for i in range(V.shape[0]):
            oi, ov = oracle32.topk(V[i], k)
            np.testing.assert_array_equal(idx[i].cpu().numpy(), oi)
            np.testing.assert_array_equal(val[i].cpu().numpy().view(np.uint32), ov.view(np.uint32))


def test_topk_static_refuses_sizes_beyond_its_scratch():
    from paper_2106_05203_b200 import binding as B
    v = torch.zeros((65, 16), dtype=torch.float32, device="cuda")
    idx = torch.zeros((65, 1), dtype=torch.int32, device="cuda")
    val = torch.zeros((65, 1), dtype=torch.float32, device="cuda")
    with pytest.raises(B.Ef21Error) as e:
        B.topk_static(v, 1, idx, val)                                   # batch > 64
    assert e.value.status == 7
    big = torch.zeros((64, (1 << 20) + 4096), dtype=torch.float32, device="cuda")
    idx = torch.zeros((64, 1), dtype=torch.int32, device="cuda")
    val = torch.zeros((64, 1), dtype=torch.float32, device="cuda")
    with pytest.raises(B.Ef21Error) as e:
        B.topk_static(big, 1, idx, val)                                 # 64 * 257 chunks > 16384
    assert e.value.status == 7
