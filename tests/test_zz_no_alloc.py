"""efcp_topk_static, the entry point that allocates nothing.

Some callers of this library cannot call cudaMalloc at the moment they need a Top-k: a
framework's memory pool may already own all free device memory, an allocation would
synchronise the whole device in the middle of their pipeline, or they run in a start-up path
that must not die with out-of-memory.  For them the library carries one fixed scratch array
and this call, which must give exactly the selection that efcp_step makes with the scratch
memory efcp_create allocates.  This file is collected last on purpose: if the added entry
point breaks, every other test has already run.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2306_06098_b200 import binding
    return binding


def selection_of_step(B, g: torch.Tensor, k: int):
    """Top-k as efcp_step makes it: first step of a fresh handle (error buffer zero, so the
    accumulator is the gradient), read back from ring slot 0."""
    h = B.Efcp(g.numel(), 1, k, 1.0)
    u = torch.empty_like(g)
    h.step(g, u)
    assert h.status() == 0
    idx, val = h.row(0)
    h.close()
    return idx, val


def test_static_topk_matches_step_selection_twice_in_a_row():
    B = _binding()
    rng = np.random.default_rng(2024)
    # the second call is smaller and tie-heavy: whatever the first left in the shared
    # scratch array must not leak into it
    cases = [(300_007, 3_001, lambda d: rng.standard_normal(d) * np.exp(rng.standard_normal(d))),
             (70_001, 7_777, lambda d: rng.integers(-2, 3, d))]
    calls_done = 0
    for d, k, make in cases:
        g = torch.from_numpy(np.ascontiguousarray(make(d), dtype=np.float32)).cuda()
        idx = torch.empty(k, dtype=torch.int32, device="cuda")
        val = torch.empty(k, dtype=torch.float32, device="cuda")
        idx.fill_(-1)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        B.topk_static(g, k, idx, val)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        if calls_done:  # (the very first call may load the library's kernels onto the device)
            assert free_after == free_before, "the call changed the device's free memory"
        calls_done += 1
        want_i, want_v = selection_of_step(B, g, k)
        got_i, got_v = idx.cpu().numpy(), val.cpu().numpy()
        assert np.array_equal(got_i, want_i)                                   # bit-exact,
        assert np.array_equal(got_v.view(np.uint32), want_v.view(np.uint32))  # as for all state
        assert np.all(np.diff(got_i) > 0)
        # and directly against the CPU oracle's Top-k (stable-sort definition)
        from oracle import ref
        ora_i, ora_v = ref.topk(g.cpu().numpy(), k)
        assert np.array_equal(got_i, ora_i)
        assert np.array_equal(got_v.view(np.uint32), ora_v.view(np.uint32))


def test_static_topk_rejects_what_it_cannot_hold():
    B = _binding()
    d = B.TOPK_STATIC_MAX_D + 1
    a = torch.zeros(d, dtype=torch.float32, device="cuda")
    idx = torch.empty(4, dtype=torch.int32, device="cuda")
    val = torch.empty(4, dtype=torch.float32, device="cuda")
    with pytest.raises(B.EfcpError) as ei:
        B.topk_static(a, 4, idx, val)
    assert ei.value.code == B.ETOOBIG
    assert "capacity" in B.strerror(B.ETOOBIG)
    with pytest.raises(B.EfcpError) as ei:
        B.topk_static(a[:8], 9, torch.empty(9, dtype=torch.int32, device="cuda"),
                      torch.empty(9, dtype=torch.float32, device="cuda"))
    assert ei.value.code == B.EINVAL
    # a vector that does not start on a 16-byte boundary (a view into a larger buffer) is
    # refused before anything is launched: the kernels would read it with vector loads
    with pytest.raises(B.EfcpError) as ei:
        B.topk_static(a[1:1001], 4, idx, val)
    assert ei.value.code == B.EINVAL
    # the largest size it accepts
    a = torch.randn(B.TOPK_STATIC_MAX_D, device="cuda")
    k = 1000
    idx = torch.empty(k, dtype=torch.int32, device="cuda")
    val = torch.empty(k, dtype=torch.float32, device="cuda")
    B.topk_static(a, k, idx, val)
    torch.cuda.synchronize()
    ref = torch.topk(a.abs(), k).indices.sort().values.to(torch.int32)
    assert torch.equal(idx, ref)  # random normals: no ties at the threshold
