"""GPU tests of the boundary itself: caller-supplied memory, the debug-checks flag, the
bounded device-side wait (failure detection without a GPU fault), device selection."""
import gc

import numpy as np
import pytest
import torch

from oracle import ref

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2306_06098_b200 import binding
    return binding


def bits(a):
    return np.ascontiguousarray(a).view(np.uint32)


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def _parity_steps(gpu, cpu, grads, d):
    g_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    u_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    for t, g in enumerate(grads):
        g_dev.copy_(torch.from_numpy(g))
        gpu.step(g_dev, u_dev)
        u_ref = cpu.step(g)
        assert gpu.status() == 0
        assert np.array_equal(bits(gpu.error()), bits(cpu.error())), t
        gi, gv = gpu.row(t % gpu.m)
        ci, cv = cpu.row(t % gpu.m)
        assert np.array_equal(gi, ci) and np.array_equal(bits(gv), bits(cv)), t
        assert rel_l2(u_dev.cpu().numpy(), u_ref) <= 1e-4


@pytest.mark.parametrize("flags,block", [(0, 0), (2, 4096), (1, 0)],
                         ids=["default", "bf16_blockwise", "rhs_accumulator"])
def test_handle_in_caller_memory_allocates_nothing(flags, block):
    """efcp_create_in carves the whole handle out of one caller-supplied buffer: the device's
    free memory must not move across create, steps and destroy, and the results are those of
    a handle that allocates for itself."""
    B = _binding()
    d, m, k, lam = 300_007, 8, 3000, 1e-3
    need = B.workspace_bytes(d, m, k, flags, block)
    assert need > 0
    if not flags and not block:
        assert need == B.state_bytes(d, m, k)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    rng = np.random.default_rng(91)
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(10)]
    g_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    u_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    warm = B.Efcp(d, m, k, lam, flags, block)  # loads every kernel of this mode once
    warm.step(g_dev.zero_(), u_dev)
    assert warm.validate() == 0 and warm.status() == 0
    warm.close()
    gc.collect()  # handles earlier tests left to the collector free their memory now, not later
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    gpu = B.Efcp(d, m, k, lam, flags, block, workspace=ws)
    cpu = ref.RefEFCP(d, m, k, lam, flags, block)
    for t, g in enumerate(grads):
        g_dev.copy_(torch.from_numpy(g))
        gpu.step(g_dev, u_dev)
        u_ref = cpu.step(g)
        free_t, _ = torch.cuda.mem_get_info()
        assert free_t >= free0, f"device memory was allocated at step {t}"
        assert np.array_equal(bits(gpu.error()), bits(cpu.error()))
        assert rel_l2(u_dev.cpu().numpy(), u_ref) <= 1e-4
    assert gpu.validate() == 0 and gpu.status() == 0
    gpu.close()
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 >= free0
    # one byte short: refused, nothing leaks
    with pytest.raises(B.EfcpError) as ei:
        B.Efcp(d, m, k, lam, flags, block, workspace=ws[:need - 256])
    assert ei.value.code == B.ENOMEM
    with pytest.raises(B.EfcpError) as ei:
        B.Efcp(d, m, k, lam, flags, block, workspace=ws[1:])  # not 256-byte aligned
    assert ei.value.code == B.EINVAL


def test_debug_checks_flag_runs_clean_and_keeps_results():
    B = _binding()
    d, m, k, lam = 200_003, 6, 2000, 1e-3
    rng = np.random.default_rng(92)
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(14)]
    gpu = B.Efcp(d, m, k, lam, B.DEBUG_CHECKS)
    cpu = ref.RefEFCP(d, m, k, lam)
    _parity_steps(gpu, cpu, grads, d)
    assert gpu.status() == 0


def test_bounded_wait_runs_out_and_the_context_survives():
    """Failure detection without a fault: under the test hook the block-wise Top-k kernel arms
    the barrier of its bulk copies but starts no copy, so nothing is in flight and its bounded
    wait simply runs out.  The step must end by itself with the sticky status EFCP_ETIMEOUT,
    the handle must be destroyable, and the device must go on working: a fresh handle then
    passes a parity case."""
    B = _binding()
    d, m, k, block = 65_536, 4, 655, 4096
    rng = np.random.default_rng(93)
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(6)]
    gpu = B.Efcp(d, m, k, 1e-3, 0, block)
    cpu = ref.RefEFCP(d, m, k, 1e-3, 0, block)
    _parity_steps(gpu, cpu, grads[:2], d)
    gpu.test_hook(B.HOOK_DROP_BLOCK_LOADS, 1)
    g_dev = torch.from_numpy(grads[2]).cuda()
    u_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    gpu.step(g_dev, u_dev)
    assert gpu.status() == B.ETIMEOUT
    assert "wait" in B.strerror(B.ETIMEOUT)
    with pytest.raises(B.EfcpError) as ei:
        gpu.error()  # state inspection reports the sticky status
    assert ei.value.code == B.ETIMEOUT
    gpu.close()
    cpu.close()
    torch.cuda.synchronize()  # the context is intact
    with pytest.raises(B.EfcpError):
        B.Efcp(d, m, k, 1e-3).test_hook(99, 1)  # unknown hook
    gpu = B.Efcp(d, m, k, 1e-3, 0, block)
    cpu = ref.RefEFCP(d, m, k, 1e-3, 0, block)
    _parity_steps(gpu, cpu, grads, d)
    assert gpu.validate() == 0
